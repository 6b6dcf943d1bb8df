// KV-block swap: pack scattered blocks (all layers, K and V) into a contiguous image and
// back.  One CTA copies one (block, layer, K|V) chunk with 16-byte accesses; the block ids
// of a launch travel in the kernel parameters, so no id array has to live on the device.
#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "internal.h"

namespace pk {

constexpr int SWAP_IDS = 512;  // block ids per launch (2 KiB of kernel parameters)
constexpr int SWAP_THREADS = 256;

struct SwapIds {
    int32_t v[SWAP_IDS];
};

struct SwapParams {
    uint8_t* k_pool;
    uint8_t* v_pool;
    uint8_t* image;           // first image slot of this launch
    int64_t layer_stride_k;   // bytes
    int64_t layer_stride_v;
    int64_t stride_block, stride_head, stride_tok;  // bytes
    int layers;
    int log2_d;               // head_dim = 1 << log2_d
    int vec_per_chunk;        // 16-byte vectors in one (block, layer, K|V) chunk
};

// OUT = true: pool -> image;  false: image -> pool
template <bool OUT>
__global__ void __launch_bounds__(SWAP_THREADS) kv_swap_kernel(const SwapParams p,
                                                               const SwapIds ids) {
    const int chunk = blockIdx.x;  // (i, layer, kv) flattened, kv fastest
    const int kv = chunk & 1;
    const int layer = (chunk >> 1) % p.layers;
    const int i = (chunk >> 1) / p.layers;
    uint8_t* pool = (kv ? p.v_pool + layer * p.layer_stride_v : p.k_pool + layer * p.layer_stride_k) +
                    (int64_t)ids.v[i] * p.stride_block;
    uint4* img = reinterpret_cast<uint4*>(p.image) + (int64_t)chunk * p.vec_per_chunk;
    const int lt = p.log2_d - 3;  // vectors per row = D / 8
    for (int v = threadIdx.x; v < p.vec_per_chunk; v += SWAP_THREADS) {
        const int dvec = v & ((1 << lt) - 1);
        const int slot = (v >> lt) & (BS - 1);
        const int head = v >> (lt + 4);
        uint4* cell = reinterpret_cast<uint4*>(pool + head * p.stride_head + slot * p.stride_tok) + dvec;
        if (OUT)
            img[v] = *cell;
        else
            *cell = img[v];
    }
}

struct SwapCall {
    const kv_pool_desc* pool;
    const pa_shape* shape;
    uint8_t* k_pool;
    uint8_t* v_pool;
    const int32_t* ids;
    int32_t n;
    uint8_t* host;
    size_t host_bytes;
    uint8_t* staging;
    size_t staging_bytes;
    cudaStream_t st;
};

static int swap_common(const SwapCall& c, bool out) {
    if (!c.pool || !c.shape) return PA_ERR_NULL;
    int rc = validate_shape(c.shape);
    if (rc) return rc;
    if (c.pool->num_layers <= 0 || c.pool->layer_stride_k < 0 || c.pool->layer_stride_v < 0 ||
        c.pool->layer_stride_k % 8 || c.pool->layer_stride_v % 8)
        return PA_ERR_SHAPE;
    if (c.n < 0) return PA_ERR_ARG;
    if (c.n == 0) return PA_OK;
    if (!c.k_pool || !c.v_pool || !c.ids || !c.host) return PA_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(c.k_pool) | reinterpret_cast<uintptr_t>(c.v_pool) |
         reinterpret_cast<uintptr_t>(c.host)) & 15)
        return PA_ERR_ALIGN;
    if (c.staging && (reinterpret_cast<uintptr_t>(c.staging) & 255)) return PA_ERR_ALIGN;

    const pa_shape& s = *c.shape;
    const size_t chunk_bytes = (size_t)s.num_kv_heads * BS * s.head_dim * 2;
    const size_t block_bytes = chunk_bytes * 2 * c.pool->num_layers;
    if (c.host_bytes < block_bytes * (size_t)c.n) return PA_ERR_HOSTBUF;

    // ids: in range, each once
    {
        std::vector<int32_t> sorted(c.ids, c.ids + c.n);
        std::sort(sorted.begin(), sorted.end());
        if (sorted.front() < 0 || sorted.back() >= s.num_blocks) return PA_ERR_BLOCK_ID;
        if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return PA_ERR_BLOCK_ID;
    }

    uint8_t* host_dev = nullptr;  // device-side address of the pinned image (direct mode)
    int per_launch = SWAP_IDS;
    if (c.staging) {
        if (c.staging_bytes < block_bytes) return PA_ERR_WORKSPACE;
        per_launch = (int)std::min<size_t>(SWAP_IDS, c.staging_bytes / block_bytes);
    } else {
        cudaPointerAttributes attr;
        rc = check_cuda(cudaPointerGetAttributes(&attr, c.host));
        if (rc) return rc;
        if (attr.type != cudaMemoryTypeHost || !attr.devicePointer) return PA_ERR_HOSTBUF;
        host_dev = static_cast<uint8_t*>(attr.devicePointer);
    }

    SwapParams p;
    p.k_pool = c.k_pool;
    p.v_pool = c.v_pool;
    p.layer_stride_k = c.pool->layer_stride_k * 2;
    p.layer_stride_v = c.pool->layer_stride_v * 2;
    p.stride_block = s.stride_block * 2;
    p.stride_head = s.stride_head * 2;
    p.stride_tok = s.stride_tok * 2;
    p.layers = c.pool->num_layers;
    p.log2_d = s.head_dim == 256 ? 8 : s.head_dim == 128 ? 7 : 6;
    p.vec_per_chunk = (int)(chunk_bytes / 16);

    // Staged swaps of more than one piece alternate between the two halves of the staging
    // buffer: the copy engine moves one half over the link (on a side stream that lives for
    // this call only) while the kernel gathers into, or scatters from, the other.  Events tie
    // the two streams together, and everything joins the caller's stream before the call
    // returns, so the caller sees ordinary stream order.
    const bool two_halves = c.staging && c.n > per_launch && c.staging_bytes / 2 >= block_bytes;
    cudaStream_t side = nullptr;
    cudaEvent_t ev_kernel[2] = {nullptr, nullptr}, ev_copy[2] = {nullptr, nullptr};
    auto cleanup = [&]() {
        for (int h = 0; h < 2; ++h) {
            if (ev_kernel[h]) cudaEventDestroy(ev_kernel[h]);
            if (ev_copy[h]) cudaEventDestroy(ev_copy[h]);
        }
        if (side) cudaStreamDestroy(side);  // work already queued on it still completes
    };
    size_t half_bytes = 0;
    if (two_halves) {
        half_bytes = (c.staging_bytes / 2) & ~(size_t)255;
        per_launch = (int)std::min<size_t>(SWAP_IDS, half_bytes / block_bytes);
        rc = check_cuda(cudaStreamCreateWithFlags(&side, cudaStreamNonBlocking));
        for (int h = 0; h < 2 && !rc; ++h) {
            rc = check_cuda(cudaEventCreateWithFlags(&ev_kernel[h], cudaEventDisableTiming));
            if (!rc) rc = check_cuda(cudaEventCreateWithFlags(&ev_copy[h], cudaEventDisableTiming));
        }
        if (rc) {
            cleanup();
            return rc;
        }
    }

    int piece = 0;
    for (int32_t done = 0; done < c.n; done += per_launch, ++piece) {
        const int m = std::min<int32_t>(per_launch, c.n - done);
        SwapIds ids;
        for (int i = 0; i < m; ++i) ids.v[i] = c.ids[done + i];
        const size_t bytes = block_bytes * (size_t)m;
        uint8_t* host_piece = c.host + block_bytes * (size_t)done;
        const unsigned grid = (unsigned)m * p.layers * 2;
        if (two_halves) {
            const int h = piece & 1;
            uint8_t* half = c.staging + (size_t)h * half_bytes;
            p.image = half;
            if (out) {
                // the half is free once the copy that emptied it two pieces ago has finished
                if (piece >= 2) rc = check_cuda(cudaStreamWaitEvent(c.st, ev_copy[h], 0));
                if (rc) break;
                kv_swap_kernel<true><<<grid, SWAP_THREADS, 0, c.st>>>(p, ids);
                count_launch();
                rc = check_cuda(cudaGetLastError());
                if (!rc) rc = check_cuda(cudaEventRecord(ev_kernel[h], c.st));
                if (!rc) rc = check_cuda(cudaStreamWaitEvent(side, ev_kernel[h], 0));
                if (!rc) rc = check_cuda(cudaMemcpyAsync(host_piece, half, bytes, cudaMemcpyDeviceToHost, side));
                if (!rc) rc = check_cuda(cudaEventRecord(ev_copy[h], side));
            } else {
                // the first copies wait for whatever the caller's stream did before this call
                // (the staging buffer may still be in use); later ones for the scatter kernel
                // that read the half two pieces ago
                if (piece < 2) {
                    rc = check_cuda(cudaEventRecord(ev_kernel[h], c.st));
                }
                if (!rc) rc = check_cuda(cudaStreamWaitEvent(side, ev_kernel[h], 0));
                if (!rc) rc = check_cuda(cudaMemcpyAsync(half, host_piece, bytes, cudaMemcpyHostToDevice, side));
                if (!rc) rc = check_cuda(cudaEventRecord(ev_copy[h], side));
                if (!rc) rc = check_cuda(cudaStreamWaitEvent(c.st, ev_copy[h], 0));
                if (rc) break;
                kv_swap_kernel<false><<<grid, SWAP_THREADS, 0, c.st>>>(p, ids);
                count_launch();
                rc = check_cuda(cudaGetLastError());
                if (!rc) rc = check_cuda(cudaEventRecord(ev_kernel[h], c.st));
            }
        } else if (c.staging) {
            p.image = c.staging;
            if (out) {
                kv_swap_kernel<true><<<grid, SWAP_THREADS, 0, c.st>>>(p, ids);
                count_launch();
                rc = check_cuda(cudaGetLastError());
                if (rc) return rc;
                rc = check_cuda(cudaMemcpyAsync(host_piece, c.staging, bytes,
                                                cudaMemcpyDeviceToHost, c.st));
            } else {
                rc = check_cuda(cudaMemcpyAsync(c.staging, host_piece, bytes,
                                                cudaMemcpyHostToDevice, c.st));
                if (rc) return rc;
                kv_swap_kernel<false><<<grid, SWAP_THREADS, 0, c.st>>>(p, ids);
                count_launch();
                rc = check_cuda(cudaGetLastError());
            }
        } else {
            p.image = host_dev + block_bytes * (size_t)done;
            if (out)
                kv_swap_kernel<true><<<grid, SWAP_THREADS, 0, c.st>>>(p, ids);
            else
                kv_swap_kernel<false><<<grid, SWAP_THREADS, 0, c.st>>>(p, ids);
            count_launch();
            rc = check_cuda(cudaGetLastError());
        }
        if (rc) break;
    }
    if (two_halves) {
        // the caller's stream continues only after the last copies of a swap-out have landed
        // (for a swap-in its own scatter kernels already come after every copy)
        if (out)
            for (int h = 0; h < 2 && h < piece; ++h) {
                const int rc2 = check_cuda(cudaStreamWaitEvent(c.st, ev_copy[h], 0));
                if (!rc) rc = rc2;
            }
        cleanup();
    }
    if (rc) return rc;
    return PA_OK;
}

}  // namespace pk

using namespace pk;

extern "C" int kv_block_bytes(const kv_pool_desc* pool, const pa_shape* shape, size_t* bytes) {
    if (!pool || !shape || !bytes) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (pool->num_layers <= 0) return PA_ERR_SHAPE;
    *bytes = (size_t)pool->num_layers * 2 * shape->num_kv_heads * BS * shape->head_dim * 2;
    return PA_OK;
}

extern "C" int kv_swap_out(const kv_pool_desc* pool, const pa_shape* shape, const void* k_pool,
                           const void* v_pool, const int32_t* block_ids, int32_t n,
                           void* pinned_host_buf, size_t host_bytes, void* staging,
                           size_t staging_bytes, void* cuda_stream) {
    SwapCall c{pool, shape, static_cast<uint8_t*>(const_cast<void*>(k_pool)),
               static_cast<uint8_t*>(const_cast<void*>(v_pool)), block_ids, n,
               static_cast<uint8_t*>(pinned_host_buf), host_bytes, static_cast<uint8_t*>(staging),
               staging_bytes, static_cast<cudaStream_t>(cuda_stream)};
    return swap_common(c, true);
}

extern "C" int kv_swap_in(const kv_pool_desc* pool, const pa_shape* shape, void* k_pool,
                          void* v_pool, const void* pinned_host_buf, size_t host_bytes,
                          const int32_t* block_ids, int32_t n, void* staging,
                          size_t staging_bytes, void* cuda_stream) {
    SwapCall c{pool, shape, static_cast<uint8_t*>(k_pool), static_cast<uint8_t*>(v_pool),
               block_ids, n, static_cast<uint8_t*>(const_cast<void*>(pinned_host_buf)), host_bytes,
               static_cast<uint8_t*>(staging), staging_bytes,
               static_cast<cudaStream_t>(cuda_stream)};
    return swap_common(c, false);
}
