// Read-bandwidth probes: what HBM delivers to a kernel that only reads, either as one long
// stream or as 4 KiB granules at scattered offsets (the access pattern of a fragmented paged
// KV pool).  They give the practical ceilings next to which the attention kernel's GB/s is
// reported.  Granules are fetched with the same mechanism the attention kernel uses: one
// bulk asynchronous copy into shared memory per granule, completion counted on an mbarrier.
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

#include "internal.h"
#include "ptx.cuh"

namespace pk {

constexpr int PROBE_WARPS = 8, PROBE_SLOTS = 6, PROBE_GRANULE = 4096;

__device__ __forceinline__ uint32_t probe_mix(uint32_t x) {
    x ^= x >> 16;
    x *= 0x7feb352du;
    x ^= x >> 15;
    x *= 0x846ca68bu;
    x ^= x >> 16;
    return x;
}

// Each warp keeps PROBE_SLOTS granules in flight in its own ring of shared-memory slots.
// scatter = 0: granule g of the buffer in order; 1: a pseudo-random permutation-like order.
__global__ void __launch_bounds__(PROBE_WARPS * 32, 1)
probe_read_kernel(const uint8_t* src, unsigned long long n_granules, int scatter, uint32_t seed,
                  unsigned long long* sink, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t slots = base + warp * PROBE_SLOTS * PROBE_GRANULE;
    const uint32_t bars = base + PROBE_WARPS * PROBE_SLOTS * PROBE_GRANULE + warp * PROBE_SLOTS * 8;
    if (lane == 0) {
        for (int s = 0; s < PROBE_SLOTS; ++s) mbar_init(bars + 8 * s, 1);
        mbar_init_fence();
    }
    __syncwarp();
    const unsigned long long total_warps = (unsigned long long)gridDim.x * PROBE_WARPS;
    const unsigned long long gw = (unsigned long long)warp * gridDim.x + blockIdx.x;
    const unsigned long long mine = n_granules > gw ? (n_granules - gw + total_warps - 1) / total_warps : 0;
    unsigned long long issued = 0, done = 0;
    uint32_t acc = 0;
    while (done < mine) {
        while (issued < mine && issued - done < PROBE_SLOTS) {
            unsigned long long g = gw + issued * total_warps;
            if (scatter) {
                // odd multiplier modulo a power of two >= n_granules, retried until in range
                unsigned long long m = 1;
                while (m < n_granules) m <<= 1;
                unsigned long long x = g;
                do {
                    x = (x * 0x9E3779B97F4A7C15ull + (seed | 1u)) & (m - 1);
                } while (x >= n_granules);
                g = x;
            }
            if (lane == 0) {
                const uint32_t s = (uint32_t)(issued % PROBE_SLOTS);
                mbar_arrive_expect_tx(bars + 8 * s, PROBE_GRANULE);
                asm volatile(
                    "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                    ::"r"(slots + s * PROBE_GRANULE), "l"(src + g * PROBE_GRANULE), "r"(PROBE_GRANULE),
                    "r"(bars + 8 * s)
                    : "memory");
            }
            ++issued;
        }
        const uint32_t s = (uint32_t)(done % PROBE_SLOTS);
        if (!mbar_wait_bounded(bars + 8 * s, (uint32_t)((done / PROBE_SLOTS) & 1), WAIT_LIMIT_NS)) {
            if (lane == 0) atomicOr(status, PA_STATUS_TIMEOUT);
            for (unsigned long long c = done + 1; c < issued; ++c)
                mbar_wait_bounded(bars + 8 * (uint32_t)(c % PROBE_SLOTS),
                                  (uint32_t)((c / PROBE_SLOTS) & 1), WAIT_LIMIT_NS);
            return;
        }
        // touch the data so that the copy is not dead: one word per lane
        uint32_t w;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(slots + s * PROBE_GRANULE + lane * 128));
        acc ^= probe_mix(w);
        __syncwarp();
        ++done;
    }
    if (acc == 0x12345678u && sink) *sink = acc;  // practically never: keeps `acc` alive
}

// Issue rate of tiled TMA loads.  `warps` warps per CTA each own a ring of PROBE_SLOTS slots;
// per iteration a warp announces one slot and `boxes` of its lanes issue one 2 KB box each
// (64 dims x 16 tokens of a [blocks][8][16][128] bf16 tensor, the K/V box of the attention
// kernels) in a single instruction, then it waits for its oldest slot.  The buffer is meant to
// fit L2 and is walked `reps` times, so what is measured is how fast boxes can be issued and
// delivered, not DRAM.
constexpr int PROBE_BOX = 2048;
__global__ void __launch_bounds__(256, 1)
probe_tma_kernel(const __grid_constant__ CUtensorMap map, unsigned n_units, int warps, int boxes,
                 int reps, unsigned* sink, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp >= warps) return;
    const uint32_t slot_bytes = (uint32_t)boxes * PROBE_BOX;
    const uint32_t slots = base + warp * PROBE_SLOTS * slot_bytes;
    const uint32_t bars = base + warps * PROBE_SLOTS * slot_bytes + warp * PROBE_SLOTS * 8;
    if (lane == 0) {
        for (int s = 0; s < PROBE_SLOTS; ++s) mbar_init(bars + 8 * s, 1);
        mbar_init_fence();
        tma_prefetch_desc(&map);
    }
    __syncwarp();
    // a unit = one (block, head) pair = two boxes; a slot takes boxes / 2 consecutive units
    const unsigned units_per_slot = (unsigned)boxes / 2;
    const unsigned n_slots = n_units / units_per_slot;   // slot-sized pieces of the buffer
    unsigned piece_mask = 1;
    while (piece_mask * 2 <= n_slots) piece_mask *= 2;
    piece_mask -= 1;
    const unsigned tw = gridDim.x * (unsigned)warps;
    const unsigned gw = (unsigned)warp * gridDim.x + blockIdx.x;
    const unsigned long long mine = (unsigned long long)((n_slots + tw - 1) / tw) * (unsigned)reps;
    unsigned long long issued = 0, done = 0;
    uint32_t acc = 0;
    while (done < mine) {
        while (issued < mine && issued - done < PROBE_SLOTS) {
            // any piece will do (the buffer is L2-resident): an odd-multiplier walk over the
            // largest power-of-two number of pieces, so that the loop holds no division
            const unsigned piece = (gw * 97u + (unsigned)issued * 1031u) & piece_mask;
            const uint32_t s = (uint32_t)(issued % PROBE_SLOTS);
            if (lane == 0) mbar_arrive_expect_tx(bars + 8 * s, slot_bytes);
            __syncwarp();
            if (lane < boxes) {
                const unsigned unit = piece * units_per_slot + (unsigned)lane / 2;
                tma_load_4d(slots + s * slot_bytes + lane * PROBE_BOX, &map, bars + 8 * s,
                            (lane & 1) * 64, 0, (int)(unit & 7u), (int)(unit >> 3));
            }
            ++issued;
        }
        const uint32_t s = (uint32_t)(done % PROBE_SLOTS);
        if (!mbar_wait_bounded(bars + 8 * s, (uint32_t)((done / PROBE_SLOTS) & 1), WAIT_LIMIT_NS)) {
            if (lane == 0) atomicOr(status, PA_STATUS_TIMEOUT);
            for (unsigned long long c = done + 1; c < issued; ++c)
                mbar_wait_bounded(bars + 8 * (uint32_t)(c % PROBE_SLOTS),
                                  (uint32_t)((c / PROBE_SLOTS) & 1), WAIT_LIMIT_NS);
            return;
        }
        uint32_t w;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(slots + s * slot_bytes + lane * 4));
        acc ^= probe_mix(w);
        __syncwarp();
        ++done;
    }
    if (acc == 0x12345678u && sink) *sink = acc;
}

}  // namespace pk

using namespace pk;

extern "C" int pa_probe_tma_issue(const void* dev_buf, size_t bytes, int32_t warps, int32_t boxes,
                                  int32_t reps, int64_t* boxes_issued, int32_t* dev_status,
                                  void* cuda_stream) {
    if (!dev_buf || !dev_status) return PA_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(dev_buf) & 255) return PA_ERR_ALIGN;
    // whole blocks of [8 heads][16 tokens][128 dims] bf16 = 32 KiB; 2 .. 16 boxes per instruction,
    // an even number (a (block, head) tile is two boxes); warps * boxes <= 16 keeps the rings
    // inside shared memory
    if (warps < 1 || warps > 8 || boxes < 2 || boxes > 16 || (boxes & 1) || warps * boxes > 16 ||
        reps < 1 || bytes < (64u << 10) || bytes > ((size_t)1 << 31))
        return PA_ERR_ARG;
    const int nb = (int)(bytes >> 15);
    pa_shape shape = {8, 8, 128, BS, nb, PA_BF16, 8 * BS * 128, BS * 128, 128};
    CUtensorMap map;
    int rc = make_cache_map(&map, dev_buf, &shape);
    if (rc) return rc;
    DeviceInfo dev;
    rc = get_device_info(&dev);
    if (rc) return rc;
    const int smem = 16 * PROBE_SLOTS * PROBE_BOX + 8 * PROBE_SLOTS * 8 + 1024;
    static std::mutex mu;
    static bool configured[64] = {false};
    {
        std::lock_guard<std::mutex> lk(mu);
        if (dev.device < 0 || dev.device >= 64) return PA_ERR_ARG;
        if (!configured[dev.device]) {
            rc = check_cuda(cudaFuncSetAttribute(
                probe_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            if (rc) return rc;
            configured[dev.device] = true;
        }
    }
    const unsigned n_units = (unsigned)nb * 8u;
    const unsigned n_slots = n_units / ((unsigned)boxes / 2);
    const unsigned tw = (unsigned)dev.sm_count * (unsigned)warps;
    if (boxes_issued)
        *boxes_issued = (int64_t)((n_slots + tw - 1) / tw) * reps * tw * boxes;
    probe_tma_kernel<<<dev.sm_count, 256, smem, static_cast<cudaStream_t>(cuda_stream)>>>(
        map, n_units, warps, boxes, reps, nullptr, dev_status);
    count_launch();
    return check_cuda(cudaGetLastError());
}

extern "C" int pa_probe_read(const void* dev_buf, size_t bytes, int32_t scattered, uint32_t seed,
                             void* dev_sink, int32_t* dev_status, void* cuda_stream) {
    if (!dev_buf || !dev_status) return PA_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(dev_buf) & 15) return PA_ERR_ALIGN;
    if (bytes < PROBE_GRANULE) return PA_ERR_ARG;
    DeviceInfo dev;
    int rc = get_device_info(&dev);
    if (rc) return rc;
    const int smem = PROBE_WARPS * PROBE_SLOTS * PROBE_GRANULE + PROBE_WARPS * PROBE_SLOTS * 8 + 128;
    // the attribute is set once per device; callers may come from several host threads
    static std::mutex mu;
    static bool configured[64] = {false};
    {
        std::lock_guard<std::mutex> lk(mu);
        if (dev.device < 0 || dev.device >= 64) return PA_ERR_ARG;
        if (!configured[dev.device]) {
            rc = check_cuda(cudaFuncSetAttribute(
                probe_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            if (rc) return rc;
            configured[dev.device] = true;
        }
    }
    probe_read_kernel<<<dev.sm_count, PROBE_WARPS * 32, smem, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const uint8_t*>(dev_buf), (unsigned long long)(bytes / PROBE_GRANULE),
        scattered ? 1 : 0, seed, static_cast<unsigned long long*>(dev_sink), dev_status);
    count_launch();
    return check_cuda(cudaGetLastError());
}
