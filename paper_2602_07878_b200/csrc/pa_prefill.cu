// Chunked causal prefill over the paged KV cache (the recomputation path of a preempted
// sequence): every query token of the chunk attends to the cached tokens up to its own
// position.  First implementation: the same independent-warp machinery as decode -- a warp
// owns 16 query rows (tokens x heads of one KV-head group) and streams the KV blocks they may
// see through its private TMA ring; neighbouring warps re-read the same blocks from L2.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "attn_block.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace pk {

enum { PF_N_GROUPS = 0, PF_COUNTER = 1, PF_STATUS = 2, PF_WORDS = 64 };

struct PrefillPlanParams {
    const int32_t* ctx_lens;
    const int32_t* cu_q_lens;
    int batch, max_blocks, total_q, tpg;  // tpg = query tokens per 16-row group
    int* hdr;
    int* gstart;  // [batch + 1] first group of each sequence
    int* status;
};

// one CTA: validate lengths, count 16-row groups per sequence, exclusive scan
__global__ void __launch_bounds__(1024, 1) pa_prefill_plan_kernel(const PrefillPlanParams p) {
    __shared__ int warp_sums[32];
    __shared__ int s_carry, s_bad;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_carry = 0, s_bad = 0;
    __syncthreads();
    for (int base = 0; base < p.batch; base += 1024) {
        const int b = base + tid;
        int n = 0;
        if (b < p.batch) {
            const int q0 = p.cu_q_lens[b], q1 = p.cu_q_lens[b + 1], L = p.ctx_lens[b];
            const int ql = q1 - q0;
            const bool ok = q0 >= 0 && ql >= 0 && q1 <= p.total_q && L >= ql &&
                            L <= p.max_blocks * BS && (b > 0 || q0 == 0);
            if (!ok) s_bad = 1;
            n = ok ? (ql + p.tpg - 1) / p.tpg : 0;
        }
        int incl = n;
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int v = warp_sums[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, v, o);
                if (lane >= o) v += u;
            }
            warp_sums[lane] = v;
        }
        __syncthreads();
        const int carry = s_carry;
        if (b < p.batch) p.gstart[b] = carry + (warp ? warp_sums[warp - 1] : 0) + incl - n;
        __syncthreads();
        if (tid == 0) s_carry = carry + warp_sums[31];
        __syncthreads();
    }
    if (tid == 0) {
        p.gstart[p.batch] = s_carry;
        p.hdr[PF_N_GROUPS] = s_carry;
        p.hdr[PF_COUNTER] = 0;
        if (s_bad) atomicOr(p.status, PA_STATUS_BAD_SEQ_LEN);
    }
}

struct PrefillParams {
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    const int32_t* block_tables;
    const int32_t* ctx_lens;
    const int32_t* cu_q_lens;
    const int* gstart;
    int* hdr;
    int* status;
    int batch, max_blocks, H, Hkv, G, NB, tpg;
    float scale_log2;
};

template <int D, int NW, int NSLOT>
__global__ void __launch_bounds__(NW * 32, 1)
pa_prefill_kernel(const __grid_constant__ CUtensorMap kmap,
                  const __grid_constant__ CUtensorMap vmap, const PrefillParams p) {
    using Frag = AttnFrag<D, true>;
    constexpr int HALVES = D / 64;
    constexpr int HALF_BYTES = BS * 128;
    constexpr int TILE = HALVES * HALF_BYTES;
    constexpr int SLOT = 2 * TILE;
    constexpr int KS = D / 16, NT = D / 8;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t slots = base + warp * (NSLOT * SLOT);
    const uint32_t bars = base + NW * NSLOT * SLOT + warp * (NSLOT * 8);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < NSLOT; ++s) mbar_init(bars + 8 * s, 1);
        mbar_init_fence();
        tma_prefetch_desc(&kmap);
        tma_prefetch_desc(&vmap);
    }
    __syncwarp();
    pdl_launch_dependents();
    pdl_wait();

    const int n_units = p.hdr[PF_N_GROUPS] * p.Hkv;
    const int G = p.G, H = p.H, Hkv = p.Hkv, tpg = p.tpg;
    const uint32_t* q32 = reinterpret_cast<const uint32_t*>(p.q);
    Frag A;
    A.init_lane(lane);
    uint32_t n_issued = 0, n_done = 0;

    while (true) {
        int w = 0;
        if (lane == 0) w = atomicAdd(&p.hdr[PF_COUNTER], 1);
        w = __shfl_sync(0xffffffffu, w, 0);
        if (w >= n_units) break;
        // later groups of a sequence see more tokens: hand the long ones out first
        const int u = n_units - 1 - w;
        const int gi = u / Hkv, kvh = u - gi * Hkv;
        int lo = 0, hi = p.batch;  // last b with gstart[b] <= gi
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (__ldg(&p.gstart[mid]) <= gi) lo = mid; else hi = mid;
        }
        const int b = lo;
        const int q0 = __ldg(&p.cu_q_lens[b]);
        const int ql = __ldg(&p.cu_q_lens[b + 1]) - q0;
        const int L = __ldg(&p.ctx_lens[b]);
        const int tok0 = (gi - __ldg(&p.gstart[b])) * tpg;  // first query token of the group
        const int ntok = min(tpg, ql - tok0);
        // rows g and g+8 of the fragment: (token, head) pairs of the group
        const int r0 = g, r1 = g + 8;
        const int tk0 = r0 / G, hd0 = r0 - tk0 * G, tk1 = r1 / G, hd1 = r1 - tk1 * G;
        const bool ok0 = tk0 < ntok, ok1 = tk1 < ntok;
        const int pos0 = L - ql + tok0 + tk0, pos1 = L - ql + tok0 + tk1;
        const int pos_max = L - ql + tok0 + ntok - 1;
        const int nblk = pos_max / BS + 1;

        uint32_t qa[KS][4];
        {
            const size_t a0 = ((size_t)(q0 + tok0 + tk0) * H + (size_t)kvh * G + hd0) * D;
            const size_t a1 = ((size_t)(q0 + tok0 + tk1) * H + (size_t)kvh * G + hd1) * D;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const size_t c = ks * 16 + 2 * t;
                qa[ks][0] = ok0 ? __ldg(&q32[(a0 + c) >> 1]) : 0u;
                qa[ks][2] = ok0 ? __ldg(&q32[(a0 + c + 8) >> 1]) : 0u;
                qa[ks][1] = ok1 ? __ldg(&q32[(a1 + c) >> 1]) : 0u;
                qa[ks][3] = ok1 ? __ldg(&q32[(a1 + c + 8) >> 1]) : 0u;
            }
        }
        A.reset();
        const int32_t* table = p.block_tables + (size_t)b * p.max_blocks;
        int ids = lane < nblk ? __ldg(&table[lane]) : 0;                 // blocks 0..31
        int ids_next = 32 + lane < nblk ? __ldg(&table[32 + lane]) : 0;  // blocks 32..63
        bool bad = false;
        int ib = 0;
        for (int cb = 0; cb < nblk; ++cb) {
            while (ib < nblk && n_issued - n_done < (uint32_t)NSLOT) {
                if (ib > 0 && (ib & 31) == 0) {
                    ids = ids_next;
                    ids_next = ib + 32 + lane < nblk ? __ldg(&table[ib + 32 + lane]) : 0;
                }
                const int id = __shfl_sync(0xffffffffu, ids, ib & 31);
                if ((unsigned)id >= (unsigned)p.NB) {
                    bad = true;
                    if (lane == 0) atomicOr(p.status, PA_STATUS_BAD_BLOCK_ID);
                }
                if (lane == 0) {
                    const uint32_t s = n_issued % NSLOT;
                    const uint32_t bar = bars + 8 * s, dst = slots + s * SLOT;
                    mbar_arrive_expect_tx(bar, SLOT);
#pragma unroll
                    for (int hf = 0; hf < HALVES; ++hf) {
                        tma_load_4d(dst + hf * HALF_BYTES, &kmap, bar, hf * 64, 0, kvh, id);
                        tma_load_4d(dst + TILE + hf * HALF_BYTES, &vmap, bar, hf * 64, 0, kvh, id);
                    }
                }
                ++n_issued;
                ++ib;
            }
            const uint32_t s = n_done % NSLOT;
            if (!mbar_wait_bounded(bars + 8 * s, (n_done / NSLOT) & 1, WAIT_LIMIT_NS)) {
                if (lane == 0) atomicOr(p.status, PA_STATUS_TIMEOUT);
                for (uint32_t c = n_done + 1; c < n_issued; ++c)
                    mbar_wait_bounded(bars + 8 * (c % NSLOT), (c / NSLOT) & 1, WAIT_LIMIT_NS);
                return;
            }
            const uint32_t kbase = slots + s * SLOT, vbase = kbase + TILE;
            const int t0 = cb * BS;
            const int lim0 = ok0 ? min(BS, max(0, pos0 + 1 - t0)) : 0;
            const int lim1 = ok1 ? min(BS, max(0, pos1 + 1 - t0)) : 0;
            A.attend(kbase, vbase, qa, lim0, lim1, min(BS, L - t0), p.scale_log2, lane);
            ++n_done;
        }
        A.reduce_row_sums();
        const float i0 = bad ? 0.f : 1.f / A.l0, i1 = bad ? 0.f : 1.f / A.l1;
        if (ok0) {
            uint32_t* dst = reinterpret_cast<uint32_t*>(
                p.out + ((size_t)(q0 + tok0 + tk0) * H + (size_t)kvh * G + hd0) * D);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
                dst[nt * 4 + t] = bad ? 0u : pack_bf16x2(A.o[nt][0] * i0, A.o[nt][1] * i0);
        }
        if (ok1) {
            uint32_t* dst = reinterpret_cast<uint32_t*>(
                p.out + ((size_t)(q0 + tok0 + tk1) * H + (size_t)kvh * G + hd1) * D);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
                dst[nt * 4 + t] = bad ? 0u : pack_bf16x2(A.o[nt][2] * i1, A.o[nt][3] * i1);
        }
    }
}

template <int D>
static int launch_prefill(const CUtensorMap& km, const CUtensorMap& vm, const PrefillParams& pp,
                          const DeviceInfo& dev, cudaStream_t st) {
    constexpr int NW = 8, NSLOT = 3 * (128 / D);
    auto kern = pa_prefill_kernel<D, NW, NSLOT>;
    const int smem = NW * NSLOT * (2 * BS * D * 2) + NW * NSLOT * 8 + 1024;
    static int configured_dev = -1;
    static std::mutex mu;
    {
        std::lock_guard<std::mutex> lk(mu);
        if (configured_dev != dev.device) {
            int rc = check_cuda(
                cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            if (rc) return rc;
            configured_dev = dev.device;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(dev.sm_count);
    cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return check_cuda(cudaLaunchKernelEx(&cfg, kern, km, vm, pp));
}

}  // namespace pk

using namespace pk;

extern "C" int pa_prefill_workspace_bytes(int32_t max_batch, size_t* bytes) {
    if (!bytes) return PA_ERR_NULL;
    if (max_batch < 0) return PA_ERR_ARG;
    *bytes = PF_WORDS * sizeof(int) + ((size_t)max_batch + 1) * sizeof(int) + 256;
    return PA_OK;
}

extern "C" int pa_prefill(const pa_shape* shape, const void* q, const void* k_cache,
                          const void* v_cache, const int32_t* block_tables,
                          int32_t max_blocks_per_seq, const int32_t* ctx_lens,
                          const int32_t* cu_q_lens, int32_t batch, int32_t total_q, float scale,
                          void* out, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                          void* cuda_stream) {
    if (!shape) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (batch < 0 || total_q < 0 || max_blocks_per_seq < 0) return PA_ERR_ARG;
    if (batch == 0 || total_q == 0) return PA_OK;
    if (!q || !k_cache || !v_cache || !block_tables || !ctx_lens || !cu_q_lens || !out || !workspace)
        return PA_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) |
         reinterpret_cast<uintptr_t>(k_cache) | reinterpret_cast<uintptr_t>(v_cache)) & 15)
        return PA_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return PA_ERR_ALIGN;
    if ((int64_t)max_blocks_per_seq * BS > INT32_MAX) return PA_ERR_ARG;
    size_t need = 0;
    pa_prefill_workspace_bytes(batch, &need);
    if (workspace_bytes < need) return PA_ERR_WORKSPACE;
    DeviceInfo dev;
    rc = get_device_info(&dev);
    if (rc) return rc;
    CUtensorMap km, vm;
    rc = make_cache_map(&km, k_cache, shape);
    if (rc) return rc;
    rc = make_cache_map(&vm, v_cache, shape);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int* hdr = static_cast<int*>(workspace);
    const int G = shape->num_q_heads / shape->num_kv_heads;

    PrefillPlanParams plan;
    plan.ctx_lens = ctx_lens;
    plan.cu_q_lens = cu_q_lens;
    plan.batch = batch;
    plan.max_blocks = max_blocks_per_seq;
    plan.total_q = total_q;
    plan.tpg = 16 / G;
    plan.hdr = hdr;
    plan.gstart = hdr + PF_WORDS;
    plan.status = dev_status ? dev_status : hdr + PF_STATUS;
    pa_prefill_plan_kernel<<<1, 1024, 0, st>>>(plan);
    count_launch();
    rc = check_cuda(cudaGetLastError());
    if (rc) return rc;

    PrefillParams pp;
    pp.q = static_cast<const __nv_bfloat16*>(q);
    pp.out = static_cast<__nv_bfloat16*>(out);
    pp.block_tables = block_tables;
    pp.ctx_lens = ctx_lens;
    pp.cu_q_lens = cu_q_lens;
    pp.gstart = plan.gstart;
    pp.hdr = hdr;
    pp.status = plan.status;
    pp.batch = batch;
    pp.max_blocks = max_blocks_per_seq;
    pp.H = shape->num_q_heads;
    pp.Hkv = shape->num_kv_heads;
    pp.G = G;
    pp.NB = shape->num_blocks;
    pp.tpg = plan.tpg;
    pp.scale_log2 = scale * 1.4426950408889634f;
    return shape->head_dim == 128 ? launch_prefill<128>(km, vm, pp, dev, st)
                                  : launch_prefill<64>(km, vm, pp, dev, st);
}
