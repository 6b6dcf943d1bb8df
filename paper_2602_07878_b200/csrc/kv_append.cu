// KV append: write each sequence's new token into its slot of one layer's paged cache.
// One thread moves 16 bytes; a (token, kv head) row of D bf16 is D/8 threads.
#include <cuda_runtime.h>

#include "internal.h"

namespace pk {

struct AppendParams {
    uint8_t* k_cache;
    uint8_t* v_cache;
    const uint4* k_new;
    const uint4* v_new;
    const int64_t* slot_mapping;
    int* status;
    int64_t stride_block, stride_head, stride_tok;  // bytes
    int64_t total_slots;
    int batch, Hkv, log2_vec;  // log2(D / 8)
};

__global__ void __launch_bounds__(256) kv_append_kernel(const AppendParams p) {
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int vec = (int)(tid & ((1 << p.log2_vec) - 1));
    const int64_t row = tid >> p.log2_vec;  // (token, kv head)
    if (row >= (int64_t)p.batch * p.Hkv) return;
    const int b = (int)(row / p.Hkv), h = (int)(row - (int64_t)b * p.Hkv);
    const int64_t slot = p.slot_mapping[b];
    if (slot < 0) return;  // padding entry
    if (slot >= p.total_slots) {
        if (vec == 0 && h == 0 && p.status) atomicOr(p.status, PA_STATUS_BAD_BLOCK_ID);
        return;
    }
    const int64_t off = (slot >> 4) * p.stride_block + h * p.stride_head + (slot & (BS - 1)) * p.stride_tok;
    reinterpret_cast<uint4*>(p.k_cache + off)[vec] = p.k_new[tid];
    reinterpret_cast<uint4*>(p.v_cache + off)[vec] = p.v_new[tid];
}

}  // namespace pk

using namespace pk;

extern "C" int kv_append(const pa_shape* shape, void* k_cache, void* v_cache, const void* k_new,
                         const void* v_new, const int64_t* slot_mapping, int32_t batch,
                         int32_t* dev_status, void* cuda_stream) {
    if (!shape) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (batch < 0) return PA_ERR_ARG;
    if (batch == 0) return PA_OK;
    if (!k_cache || !v_cache || !k_new || !v_new || !slot_mapping) return PA_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(k_cache) | reinterpret_cast<uintptr_t>(v_cache) |
         reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new)) & 15)
        return PA_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(slot_mapping) & 7) return PA_ERR_ALIGN;
    AppendParams p;
    p.k_cache = static_cast<uint8_t*>(k_cache);
    p.v_cache = static_cast<uint8_t*>(v_cache);
    p.k_new = static_cast<const uint4*>(k_new);
    p.v_new = static_cast<const uint4*>(v_new);
    p.slot_mapping = slot_mapping;
    p.status = dev_status;
    p.stride_block = shape->stride_block * 2;
    p.stride_head = shape->stride_head * 2;
    p.stride_tok = shape->stride_tok * 2;
    p.total_slots = (int64_t)shape->num_blocks * BS;
    p.batch = batch;
    p.Hkv = shape->num_kv_heads;
    p.log2_vec = shape->head_dim == 256 ? 5 : shape->head_dim == 128 ? 4 : 3;
    const int64_t threads = (int64_t)batch * p.Hkv << p.log2_vec;
    const unsigned grid = (unsigned)((threads + 255) / 256);
    kv_append_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(p);
    count_launch();
    return check_cuda(cudaGetLastError());
}
