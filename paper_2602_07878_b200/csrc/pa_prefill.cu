// Chunked causal prefill over the paged KV cache (the recomputation path of a preempted
// sequence): every query token of the chunk attends to the cached tokens up to its own
// position.  Two implementations behind pa_prefill / pa_prefill_split:
//   * pa_prefill_tc_kernel: tcgen05 tensor cores, 128-row tiles, scores, weights and output
//     accumulator in tensor memory, optionally the KV range of a tile split over CTAs, the
//     last of which to finish combines the partial rows (every supported shape);
//   * pa_prefill_kernel: the independent-warp machinery of decode -- a warp owns 16 query rows
//     (tokens x heads of one KV-head group) and streams the KV blocks they may see through
//     its private TMA ring; selected with PAGEDKV_PREFILL=mma, kept as a second implementation.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <mutex>
#include <string>
#include <type_traits>

#include "attn_block.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace pk {

enum { PF_N_GROUPS = 0, PF_COUNTER = 1, PF_STATUS = 2, PF_WORDS = 64 };

struct PrefillPlanParams {
    const int32_t* ctx_lens;
    const int32_t* cu_q_lens;
    int batch, max_blocks, total_q, tpg;  // tpg = query tokens per 16-row group
    int split_steps;  // KV range of one unit in 64-token steps (0 = the whole context)
    int* hdr;
    int* gstart;  // [batch + 1] first group of each sequence
    int* status;
};

// number of KV splits of a sequence with L cached tokens when a unit covers T 64-token steps
__host__ __device__ __forceinline__ int kv_splits(int L, int T) {
    if (T <= 0 || L <= 0) return 1;
    const int steps = (L - 1) / 64 + 1;
    return (steps + T - 1) / T;
}

// one CTA: validate lengths, count units (row groups x KV splits) per sequence, exclusive scan
__global__ void __launch_bounds__(1024, 1) pa_prefill_plan_kernel(const PrefillPlanParams p) {
    __shared__ int warp_sums[32];
    __shared__ int s_carry, s_bad;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_carry = 0, s_bad = 0;
    pdl_launch_dependents();
    pdl_wait();  // the lengths may come from the kernel before; the header is still being read
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
            n = ok ? (ql + p.tpg - 1) / p.tpg * kv_splits(L, p.split_steps) : 0;
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
    constexpr int NW = D == 256 ? 4 : 8, NSLOT = D == 64 ? 6 : 3;
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


// ======================================================================================
// tcgen05 version: a row tile = 128 query rows ((token, head) pairs of one KV-head group)
// ======================================================================================
// Warps 0 .. 4 NT - 1: softmax and epilogue, four per tile (thread i of a tile's warps owns
// row i = TMEM lane i); then four TMA producer warps and one MMA warp.  Per 64-token KV step and
// tile: S = Q K^T (M 128, N 64, K head_dim) into one of two TMEM score buffers, the softmax
// warps turn S into bf16 weights P written back over the first 32 columns of that score
// buffer (and rescale the TMEM accumulator O when a row maximum has grown by more than 2^8),
// then O += P V (M 128, N head_dim, K 64) with P read from tensor memory: the weights never
// touch shared memory, whose bandwidth the MMAs' operand reads already fill.  Two score
// buffers and a ring of K/V tiles let Q K^T of step j+1 overlap the softmax of step j.
namespace tc {
constexpr int ROWS = 128, STEP = 64;
// Of every 8 pairs of weights, how many take the packed cubic on the FMA pipe instead of EX2.
// With one TMA producer warp the special-function unit was the scarcer resource and 2 was
// best; since the K/V feed keeps up, the softmax warps are bound by instruction issue and the
// cubic's extra instructions cost more than they save (512-token recompute leg: 1110 TFLOP/s
// at 0, 1103 at 1, 1083 at 2, 1057 at 3, 1012 at 4).
#ifndef PAGEDKV_POLY_PAIRS
#define PAGEDKV_POLY_PAIRS 0
#endif
constexpr int POLY_PAIRS = PAGEDKV_POLY_PAIRS;
constexpr int GROUP_BYTES = STEP * 128;  // one 64-dim column group of a 64-token K or V tile
// D = head_dim (64, 128, 256); NT = row tiles per CTA (two tiles = two softmax warpgroups
// taking turns on the tensor pipe and sharing the K/V rings).
template <int D, int NT>
struct Cfg {
    static constexpr int NG = D / 64;                     // 64-dim column groups
    static constexpr int Q_GROUP = ROWS * 128;            // one column group of a Q tile
    static constexpr int Q_BYTES = NG * Q_GROUP;
    static constexpr int TILE_BYTES = NG * GROUP_BYTES;   // K (or V) of one 64-token step
    // Head_dim 64 and 128: four stages, K and V of a step signalled and released together
    // (one barrier test and one commit less per step for the MMA warp).  Head_dim 256 (64 KB
    // of Q, 32 KB per tile) has room for five tiles only: K, free again once Q K^T of its
    // step has run, gets two, V, needed until P V, gets three (measured: the other way round
    // is 1.6 times slower), each ring with its own barriers.
    static constexpr bool SPLIT_RINGS = D == 256;
    static constexpr int KS = SPLIT_RINGS ? 2 : 4, VS = SPLIT_RINGS ? 3 : 4;
    static constexpr int OFF_Q = 0, OFF_K = NT * Q_BYTES, OFF_V = OFF_K + KS * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_V + VS * TILE_BYTES;
    // barriers (8 bytes each): shared ones, then eight per tile
    static constexpr int B_QFULL = 0, B_KFULL = 1, B_KEMPTY = B_KFULL + KS, B_VFULL = B_KEMPTY + KS,
                         B_VEMPTY = B_VFULL + VS, B_TILE = B_VEMPTY + VS;
    static constexpr int B_COUNT = B_TILE + 8 * NT;
    static constexpr int OFF_MISC = OFF_BAR + B_COUNT * 8;  // tmem base, abort flag, bad flag
    static constexpr int SMEM_BYTES = OFF_MISC + 64 + 1024;  // + slack for 1024-byte alignment
    // per tile: S0 [0,64) S1 [64,128) O [128,128+D); P of step j lies over S(j % 2) [0,32)
    static constexpr int TILE_COLS = 2 * STEP + D;
    static constexpr int TMEM_COLS = NT * TILE_COLS <= 256 ? 256 : 512;
    static_assert(NT * TILE_COLS <= 512, "tensor memory holds 512 columns");
    static_assert(SMEM_BYTES <= 232448, "shared memory of one CTA");
    // Four TMA producer warps, one per 16-token block of a step: a single warp delivers a 2 KB
    // box about every 85 cycles however many are in flight (pa_probe_tma_issue), so one warp
    // issuing the 16 boxes of a head_dim-128 step cannot keep up with the MMAs; four warps
    // with four boxes each take half the time.
    static constexpr int N_PRODUCERS = 4;
    static constexpr int PRODUCER_WARP = 4 * NT, MMA_WARP = 4 * NT + N_PRODUCERS,
                         THREADS = (4 * NT + N_PRODUCERS + 1) * 32;
};
// per-tile barrier indices, relative to Cfg::B_TILE + 8 * tile
enum { T_SFULL = 0, T_PFULL = 2, T_PVDONE = 4 };
}  // namespace tc

struct PrefillTcParams {
    PrefillParams base;
    int tokens_per_tile;  // 128 / G, rounded down: rows tokens_per_tile * G .. 127 of a tile are idle
    // KV split: a unit covers `split_steps` 64-token steps of its tile's visible context (0 =
    // all of it).  The units of one row group (same query tokens, same KV head) each leave a
    // partial record -- per row the reference exponent and weight sum (a negative sum marks a
    // split that met a bad block id) and the un-normalised fp32 output row -- and count
    // themselves in; the one that arrives last merges the records into the output rows.
    // Records are laid out for threads that own a row each:
    //   part_ml[((group * split_cap + split) * NT + tile) * 128 + row]              float2
    //   part_o [(((group * split_cap + split) * NT + tile) * D/4 + chunk) * 128 + row]  float4
    // group = ((q0 + tok0) / tokens per CTA + sequence) * Hkv + KV head.
    int split_steps, split_cap;
    float* part_ml;
    float* part_o;
    // arrive[group]: (epoch << 8) | units arrived in the call numbered `epoch` on this
    // workspace; a word from another call counts as zero, so nothing needs resetting
    int* arrive;
    int epoch;
    // Batches of at most 32 sequences need no plan kernel: every CTA validates the lengths and
    // scans the unit counts itself (one warp, a few hundred cycles) and only CTA 0 reports.
    int fold_plan, total_q;
};

// The merge of a row group by its last unit, two to four splits (the usual case):
//   out = sum_s 2^(m_s - M) o_s / sum_s 2^(m_s - M) l_s.
template <int D, int NT>
__device__ __forceinline__ void merge_few_splits(int n_vis, int split, float m_ref, float l,
                                              bool bad_own, const float2* ml_all,
                                              const float4* o_all, size_t rec0, int row,
                                              bool row_ok, __nv_bfloat16* dst, uint32_t tcol,
                                              uint32_t lane_base) {
    using namespace tc;
    // The last unit of the row group, two to four splits (the usual case):
    //   out = sum_s 2^(m_s - M) o_s / sum_s 2^(m_s - M) l_s.
    // Its own row is still in tensor memory; the pairs of the other splits come in
    // one round trip, their rows 32 floats at a time with the loads of two splits
    // in flight together.
    __threadfence();
    float2 ml[4];
#pragma unroll
    for (int sp = 0; sp < 4; ++sp) {
        ml[sp] = make_float2(-INFINITY, 0.f);
        if (sp == split) ml[sp] = make_float2(m_ref, bad_own ? -1.f : l);
        else if (sp < n_vis && row_ok)
            ml[sp] = __ldcg(&ml_all[(rec0 + (size_t)sp * NT) * 128 + row]);
    }
    const float M = fmaxf(fmaxf(ml[0].x, ml[1].x), fmaxf(ml[2].x, ml[3].x));
    const bool bad = ml[0].y < 0.f || ml[1].y < 0.f || ml[2].y < 0.f || ml[3].y < 0.f;
    float w[4], lsum = 0.f;
#pragma unroll
    for (int sp = 0; sp < 4; ++sp) {
        w[sp] = ml[sp].x == -INFINITY ? 0.f : ex2(ml[sp].x - M);
        lsum = fmaf(w[sp], ml[sp].y, lsum);
    }
    const float inv = (bad || !(lsum > 0.f)) ? 0.f : 1.f / lsum;
    float w_own = 0.f;
#pragma unroll
    for (int sp = 0; sp < 4; ++sp) {
        w[sp] *= inv;
        if (sp == split) w_own = w[sp];
    }
    // the other splits, in ascending order (at most three)
    int oth[3] = {0, 0, 0};
    {
        int k = 0;
#pragma unroll
        for (int sp = 0; sp < 4; ++sp)
            if (sp != split && sp < n_vis && k < 3) oth[k++] = sp;
    }
    const int n_oth = n_vis - 1;
    auto w_of = [&](int sp) { return sp == 0 ? w[0] : sp == 1 ? w[1] : sp == 2 ? w[2] : w[3]; };
#pragma unroll 1
    for (int c = 0; c < D; c += 32) {
        uint32_t o[32];
        tmem_ld32(tcol + lane_base + 2 * STEP + c, o);
        float4 x0[8], x1[8];
        const float4* s0 = o_all + ((rec0 + (size_t)oth[0] * NT) * (D / 4) + (c >> 2)) * 128 + row;
        const float4* s1 = o_all + ((rec0 + (size_t)oth[1] * NT) * (D / 4) + (c >> 2)) * 128 + row;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            x0[i] = n_oth > 0 && row_ok ? __ldcg(s0 + (size_t)i * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
            x1[i] = n_oth > 1 && row_ok ? __ldcg(s1 + (size_t)i * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        tmem_wait_ld();
        // The weighted rows are added in the order of their splits, whichever unit
        // does the adding: the result does not depend on which one arrived last.
        float acc[32];
        const float wa = n_oth > 0 ? w_of(oth[0]) : 0.f, wb = n_oth > 1 ? w_of(oth[1]) : 0.f;
        const bool own_first = split <= 1;  // this unit's row is among the first two terms
        const float* xa = reinterpret_cast<const float*>(x0);
        const float* xb = reinterpret_cast<const float*>(x1);
        if (n_oth <= 2) {
            // two or three splits: one fused chain in split order (the branch is
            // the same for every thread of the CTA)
            if (split == 0) {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    acc[e] = fmaf(wb, xb[e], fmaf(wa, xa[e], w_own * __uint_as_float(o[e])));
            } else if (split == 1) {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    acc[e] = fmaf(wb, xb[e], fmaf(w_own, __uint_as_float(o[e]), wa * xa[e]));
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    acc[e] = fmaf(w_own, __uint_as_float(o[e]), fmaf(wb, xb[e], wa * xa[e]));
            }
        } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const float pa = w_own * __uint_as_float(o[e]);
                const float pb = wa * xa[e], pc = wb * xb[e];
                acc[e] = own_first ? (pa + pb) + pc : pb + pc;
            }
        }
        if (n_oth > 2) {
            const float4* s2 = o_all + ((rec0 + (size_t)oth[2] * NT) * (D / 4) + (c >> 2)) * 128 + row;
            const float wc = w_of(oth[2]);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 x = row_ok ? __ldcg(s2 + (size_t)i * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
                const float xd[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float pa = w_own * __uint_as_float(o[4 * i + e]), pd = wc * xd[e];
                    float& t = acc[4 * i + e];
                    t = own_first ? t + pd : split == 2 ? (t + pa) + pd : (t + pd) + pa;
                }
            }
        }
        if (row_ok) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
                uint4 w4;
                w4.x = bad ? 0u : pack_bf16x2(acc[i], acc[i + 1]);
                w4.y = bad ? 0u : pack_bf16x2(acc[i + 2], acc[i + 3]);
                w4.z = bad ? 0u : pack_bf16x2(acc[i + 4], acc[i + 5]);
                w4.w = bad ? 0u : pack_bf16x2(acc[i + 6], acc[i + 7]);
                *reinterpret_cast<uint4*>(dst + c + i) = w4;
            }
        }
    }
}

template <int D, int NT>
__global__ void __launch_bounds__(tc::Cfg<D, NT>::THREADS, 1)
pa_prefill_tc_kernel(const __grid_constant__ CUtensorMap qmap,
                     const __grid_constant__ CUtensorMap kmap,
                     const __grid_constant__ CUtensorMap vmap, const PrefillTcParams tp) {
    using namespace tc;
    using C = Cfg<D, NT>;
    constexpr int NG = C::NG, KS = C::KS, VS = C::VS, Q_BYTES = C::Q_BYTES, TILE_BYTES = C::TILE_BYTES;
    constexpr int OFF_Q = C::OFF_Q, OFF_K = C::OFF_K, OFF_V = C::OFF_V;
    constexpr int OFF_BAR = C::OFF_BAR, OFF_MISC = C::OFF_MISC, TMEM_COLS = C::TMEM_COLS;
    constexpr int TILE_COLS = C::TILE_COLS;
    constexpr int B_QFULL = C::B_QFULL, B_KFULL = C::B_KFULL, B_KEMPTY = C::B_KEMPTY;
    constexpr int B_VFULL = C::SPLIT_RINGS ? C::B_VFULL : C::B_KFULL, B_VEMPTY = C::B_VEMPTY;
    constexpr bool SPLIT = C::SPLIT_RINGS;  // without it B_VFULL is B_KFULL and B_KEMPTY is unused
    const PrefillParams& p = tp.base;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (sbase - smem_u32(smem_raw));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    auto bar = [&](int i) { return sbase + OFF_BAR + 8 * i; };
    volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(gbase + OFF_MISC);
    // misc[0] = TMEM base address, misc[1] = abort flag, misc[2] = bad block id seen,
    // misc[3] = this unit is the last of its row group to arrive

    // Dependents (the next call) start once every CTA here has passed the
    // wait, i.e. when all that precedes this call in the stream is complete: they may then read
    // the call's inputs before they wait for this grid themselves.
    pdl_wait();
    pdl_launch_dependents();

    // ---- which tile -------------------------------------------------------------------------
    const int G = p.G, H = p.H, Hkv = p.Hkv, tpt = tp.tokens_per_tile;
    __shared__ int s_gstart[33];
    const int* gs = p.gstart;
    if (tp.fold_plan) {  // the plan kernel's work for a small batch (same checks, same counts)
        if (warp == 0) {
            int n = 0;
            bool bad = false;
            if (lane < p.batch) {
                const int q0 = p.cu_q_lens[lane], q1 = p.cu_q_lens[lane + 1], L = p.ctx_lens[lane];
                const int ql = q1 - q0;
                const bool ok = q0 >= 0 && ql >= 0 && q1 <= tp.total_q && L >= ql &&
                                L <= p.max_blocks * BS && (lane > 0 || q0 == 0);
                bad = !ok;
                n = ok ? (ql + p.tpg - 1) / p.tpg * kv_splits(L, tp.split_steps) : 0;
            }
            int incl = n;
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            s_gstart[lane + 1] = incl;
            if (lane == 0) s_gstart[0] = 0;
            if (blockIdx.x == 0 && __any_sync(0xffffffffu, bad) && lane == 0)
                atomicOr(p.status, PA_STATUS_BAD_SEQ_LEN);
        }
        __syncthreads();
        gs = s_gstart;
    }
    const int n_units = (tp.fold_plan ? s_gstart[p.batch] : p.hdr[PF_N_GROUPS]) * Hkv;
    if ((int)blockIdx.x >= n_units) return;
    const int u = n_units - 1 - blockIdx.x;  // later tiles see more tokens: start them first
    const int gi = u / Hkv, kvh = u - gi * Hkv;
    int lo = 0, hi = p.batch;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (gs[mid] <= gi) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int q0 = p.cu_q_lens[b], ql = p.cu_q_lens[b + 1] - q0, L = p.ctx_lens[b];
    const int n_split = kv_splits(L, tp.split_steps);   // units per row group of this sequence
    // Units of a sequence in launch order (blockIdx ascending = u descending): split 0 of every
    // row group, later row groups first, then split 1, ...  The last split is the short one
    // when the split length does not divide the context, and short units fill the SMs last.
    const int r = gi - gs[b];
    const int n_groups_b = (ql + p.tpg - 1) / p.tpg;    // row groups (CTAs per split) of this sequence
    const int split = n_split - 1 - r / n_groups_b;
    const int tok0 = (r % n_groups_b) * (NT * tpt);     // first query token of the CTA
    const int ntok_cta = min(NT * tpt, ql - tok0);
    const int pos_max = L - ql + tok0 + ntok_cta - 1;
    const int j0 = split * tp.split_steps;              // first 64-token step of this unit
    const int n_steps = min(pos_max / STEP + 1 - j0, n_split > 1 ? tp.split_steps : 0x7fffffff);
    if (n_steps <= 0) return;                           // the tile sees nothing of this split
    const int nblk_seq = (L + BS - 1) / BS;
    // the row group's index among all row groups of the call (see PrefillTcParams), and the
    // number of splits whose units exist for it: those that start at or before its last position
    const int group = ((q0 + tok0) / (NT * tpt) + b) * Hkv + kvh;
    const int n_vis = min(n_split, (pos_max / STEP + 1 + tp.split_steps - 1) / max(tp.split_steps, 1));
    const int rows_used = tpt * G;                      // < 128 when G does not divide 128

    if (tid == 0) {
        mbar_init(bar(B_QFULL), 1);
        // a K/V stage is full once each producer warp has announced and delivered its block
        for (int i = 0; i < KS; ++i)
            mbar_init(bar(B_KFULL + i), C::N_PRODUCERS), mbar_init(bar(B_KEMPTY + i), 1);
        for (int i = 0; i < VS; ++i)
            mbar_init(bar(B_VFULL + i), C::N_PRODUCERS), mbar_init(bar(B_VEMPTY + i), 1);
        for (int t = 0; t < NT; ++t)
            for (int i = 0; i < 2; ++i) {
                mbar_init(bar(C::B_TILE + 8 * t + T_SFULL + i), 1);
                mbar_init(bar(C::B_TILE + 8 * t + T_PFULL + i), 4);
                mbar_init(bar(C::B_TILE + 8 * t + T_PVDONE + i), 1);
            }
        mbar_init_fence();
        misc[1] = 0;
        misc[2] = 0;
    }
    // rows of the Q tiles that no (token, head) pair maps to are never loaded: give them zeros
    if (rows_used < ROWS && warp < 4 * NT) {
        const int ti = warp >> 2, row = (warp & 3) * 32 + lane;
        if (row >= rows_used)
            for (int g = 0; g < NG; ++g)
                for (int c = 0; c < 8; ++c)
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(
                                     sbase + OFF_Q + ti * Q_BYTES + g * C::Q_GROUP + row * 128 + c * 16),
                                 "r"(0u)
                                 : "memory");
        fence_proxy_async_smem();
    }
    if (warp == C::MMA_WARP) tmem_alloc(sbase + OFF_MISC, TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = misc[0];

    // every wait is bounded; a wait that gives up raises the abort flag and everyone leaves
    auto wait = [&](int b_idx, uint32_t parity) -> bool {
        if (mbar_try_wait(bar(b_idx), parity)) return true;
        if (misc[1]) return false;
        if (mbar_wait_bounded(bar(b_idx), parity, WAIT_LIMIT_NS)) return true;
        misc[1] = 1;
        atomicOr(p.status, PA_STATUS_TIMEOUT);
        return false;
    };

    if (warp >= C::PRODUCER_WARP && warp < C::PRODUCER_WARP + C::N_PRODUCERS) {
        // ===================== TMA producers =====================
        // Warp pw fetches block pw of every 64-token step: its K boxes and its V boxes, one box
        // (64 dims x 16 tokens) per lane.
        const int pw = warp - C::PRODUCER_WARP;
        if (pw == 0 && lane == 0) {
            tma_prefetch_desc(&qmap);
            mbar_arrive_expect_tx(bar(B_QFULL), NT * NG * rows_used * 128);
            for (int t = 0; t < NT; ++t)  // tile t holds query tokens tok0 + t * tpt ..
                for (int g = 0; g < NG; ++g)
                    tma_load_4d(sbase + OFF_Q + t * Q_BYTES + g * C::Q_GROUP, &qmap, bar(B_QFULL),
                                g * 64, 0, kvh, q0 + tok0 + t * tpt);
        }
        if (lane == 0) {
            tma_prefetch_desc(&kmap);
            tma_prefetch_desc(&vmap);
        }
        const int32_t* table = p.block_tables + (size_t)b * p.max_blocks;
        // block ids are fetched 32 at a time, one window ahead; the unit starts at block 4 * j0
        const int win0 = (j0 * 4) & ~31;
        int ids = win0 + lane < nblk_seq ? __ldg(&table[win0 + lane]) : p.NB;
        int ids_next = win0 + 32 + lane < nblk_seq ? __ldg(&table[win0 + 32 + lane]) : p.NB;
        // shared rings: lanes [0, NG) take the K boxes, [NG, 2 NG) the V boxes, one instruction;
        // split rings: lanes [0, NG) issue K, then V, each against its own barrier
        const bool is_v = !SPLIT && lane >= NG;
        const int grp = is_v ? lane - NG : lane;
        const uint32_t tile_off = grp * GROUP_BYTES + pw * (BS * 128);
        constexpr uint32_t BLOCK_BYTES = TILE_BYTES / 4;  // K (or V) of one block, all column groups
        for (int j = 0; j < n_steps; ++j) {
            const int blk0 = (j0 + j) * 4;
            if (blk0 > win0 && (blk0 & 31) == 0) {
                ids = ids_next;
                ids_next = blk0 + 32 + lane < nblk_seq ? __ldg(&table[blk0 + 32 + lane]) : p.NB;
            }
            const int id = __shfl_sync(0xffffffffu, ids, (blk0 + pw) & 31);
            const bool used = blk0 + pw < nblk_seq;
            if (lane == 0 && used && (unsigned)id >= (unsigned)p.NB) {
                misc[2] = 1;
                atomicOr(p.status, PA_STATUS_BAD_BLOCK_ID);
            }
            // an id outside the pool is out of the tensor's bounds and reads as zeros
            const int coord = used ? id : p.NB;
            const int ks = j % KS, vs = j % VS;
            if (SPLIT) {
                if (j >= KS && !wait(B_KEMPTY + ks, ((j / KS) - 1) & 1)) break;
                if (lane == 0) mbar_arrive_expect_tx(bar(B_KFULL + ks), BLOCK_BYTES);
                __syncwarp();
                if (lane < NG)
                    tma_load_4d(sbase + OFF_K + ks * TILE_BYTES + tile_off, &kmap, bar(B_KFULL + ks),
                                grp * 64, 0, kvh, coord);
                if (j >= VS && !wait(B_VEMPTY + vs, ((j / VS) - 1) & 1)) break;
                if (lane == 0) mbar_arrive_expect_tx(bar(B_VFULL + vs), BLOCK_BYTES);
                __syncwarp();
                if (lane < NG)
                    tma_load_4d(sbase + OFF_V + vs * TILE_BYTES + tile_off, &vmap, bar(B_VFULL + vs),
                                grp * 64, 0, kvh, coord);
            } else {
                if (j >= VS && !wait(B_VEMPTY + vs, ((j / VS) - 1) & 1)) break;
                if (lane == 0) mbar_arrive_expect_tx(bar(B_KFULL + ks), 2 * BLOCK_BYTES);
                __syncwarp();
                if (lane < 2 * NG)
                    tma_load_4d(sbase + (is_v ? OFF_V + vs * TILE_BYTES : OFF_K + ks * TILE_BYTES) + tile_off,
                                is_v ? &vmap : &kmap, bar(B_KFULL + ks), grp * 64, 0, kvh, coord);
            }
        }
    } else if (warp == C::MMA_WARP) {
        // ===================== MMA issuer =====================
        // The whole warp walks the loop and one elected lane issues: descriptor arithmetic
        // that is uniform across the warp stays off the issuing lane's critical path (issued
        // from a single-lane branch an MMA costs 50-65 cycles of issue, this way 30-40).
        // Per step j and tile: Q K^T of step j, then P V of step j-1, so that the wait for the
        // weights comes while the tensor pipe still has the Q K^T just issued in its queue.
        // S(j % 2) is free for Q K^T of step j once P V of step j-2, which read its weights
        // from there, has been issued: MMAs of one thread execute in issue order.
        constexpr uint32_t idesc_qk = tc_idesc_bf16(ROWS, STEP, false);
        constexpr uint32_t idesc_pv = tc_idesc_bf16(ROWS, D, true);
        auto wait_all = [&](int b_idx, uint32_t parity) -> bool {
            return __all_sync(0xffffffffu, wait(b_idx, parity));
        };
        // This warp shares its scheduler with two softmax warps, so the loop is kept short:
        // descriptors are the three bases below plus constants in the address field (an
        // address inside this CTA's shared memory never carries out of its 14 bits).
        const bool leader = elect_one();
        const uint64_t q_desc = tc_smem_desc(sbase + OFF_Q, 16, 1024);
        const uint64_t k_desc0 = tc_smem_desc(sbase + OFF_K, 16, 1024);
        const uint64_t v_desc0 = tc_smem_desc(sbase + OFF_V, GROUP_BYTES, 1024);
        // A barrier test is a shared-memory access that queues behind the MMAs' operand reads
        // (150-200 cycles under load), so every barrier is tested once ahead of time and the
        // answer is looked at only after the MMAs in between have been issued; the full wait
        // runs only when that early test failed.
        bool ok = wait_all(B_QFULL, 0) && wait_all(B_KFULL, 0);
        for (int j = 0; ok && j <= n_steps; ++j) {
            const int i = j - 1;  // the step whose P V is issued in this iteration
            const int ks = j % KS, vs = (j + VS - 1) % VS;
            const bool k_next_early =
                j + 1 < n_steps ? mbar_try_wait(bar(B_KFULL + (j + 1) % KS), ((j + 1) / KS) & 1) : true;
            const bool v_early =
                SPLIT && j >= 1 ? mbar_try_wait(bar(B_VFULL + vs), (i / VS) & 1) : true;
            const uint64_t k_desc = k_desc0 + (uint64_t)(ks * (TILE_BYTES >> 4));
            const uint64_t v_desc = v_desc0 + (uint64_t)(vs * (TILE_BYTES >> 4));
            const uint32_t s_col = tmem + (j & 1) * STEP, p_col = tmem + ((j + 1) & 1) * STEP;
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                const int tb = C::B_TILE + 8 * t;
                const bool p_early =
                    j >= 1 ? mbar_try_wait(bar(tb + T_PFULL + (i & 1)), (i >> 1) & 1) : true;
                if (j < n_steps) {  // S[t][j % 2] = Q_t K_j^T
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint64_t a =
                            q_desc + (uint64_t)((t * Q_BYTES + (kk >> 2) * C::Q_GROUP + (kk & 3) * 32) >> 4);
                        const uint64_t bd = k_desc + (uint64_t)(((kk >> 2) * GROUP_BYTES + (kk & 3) * 32) >> 4);
                        if (leader) tc_mma_bf16(s_col + t * TILE_COLS, a, bd, idesc_qk, kk > 0);
                    }
                    if (leader) tc_commit(bar(tb + T_SFULL + (j & 1)));
                    // the last tile's Q K^T was the last reader of this step's K
                    if (SPLIT && t == NT - 1 && leader) tc_commit(bar(B_KEMPTY + ks));
                }
                if (j >= 1) {  // O[t] += P_{j-1} V_{j-1}
                    if (SPLIT && t == 0 && !__all_sync(0xffffffffu, v_early)) {
                        ok = wait_all(B_VFULL + vs, (i / VS) & 1);
                        if (!ok) break;
                    }
                    if (!__all_sync(0xffffffffu, p_early)) {
                        ok = wait_all(tb + T_PFULL + (i & 1), (i >> 1) & 1);
                        if (!ok) break;
                    }
                    tc_fence_after_sync();
#pragma unroll
                    for (int kk = 0; kk < STEP / 16; ++kk) {
                        // V is MN-major: 64-dim column groups GROUP_BYTES apart, 8-token groups
                        // 1 KiB apart; 16 tokens (2 KiB) per MMA
                        const uint64_t bd = v_desc + (uint64_t)((kk * 16 * 128) >> 4);
                        if (leader)
                            tc_mma_bf16_ta(tmem + t * TILE_COLS + 2 * STEP, p_col + t * TILE_COLS + kk * 8,
                                           bd, idesc_pv, (i > 0 || kk > 0) ? 1u : 0u);
                    }
                    if (leader) tc_commit(bar(tb + T_PVDONE + (i & 1)));
                }
            }
            if (!ok) break;
            // every tile's P V of the previous step is queued: its V tile (without split rings,
            // its K tile too) may be refilled
            if (j >= 1 && leader) tc_commit(bar(B_VEMPTY + vs));
            if (j + 1 < n_steps && !__all_sync(0xffffffffu, k_next_early))
                ok = wait_all(B_KFULL + (j + 1) % KS, ((j + 1) / KS) & 1);
        }
    } else {
        // ===================== softmax + epilogue: thread = row =====================
        const int ti = warp >> 2;                       // row tile of this warpgroup
        const int row = (warp & 3) * 32 + lane;
        const int tk = row / G, hd = row - tk * G;
        const int qtok = tok0 + ti * tpt + tk;          // query token within the sequence's chunk
        const bool row_ok = row < rows_used && qtok < ql;  // idle rows exist when G does not divide 128
        const int pos = row_ok ? L - ql + qtok : 0x7fffffff;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tcol = tmem + ti * TILE_COLS;    // this tile's S0, S1, O columns
        const int tb = C::B_TILE + 8 * ti;              // this tile's barriers
        const float sl2 = p.scale_log2;
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_steps; ++j) {
            ok = wait(tb + T_SFULL + (j & 1), (j >> 1) & 1);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sr[2][32];
            tmem_ld32(tcol + lane_base + (j & 1) * STEP, sr[0]);
            tmem_ld32(tcol + lane_base + (j & 1) * STEP + 32, sr[1]);
            tmem_wait_ld();

            const int t0 = (j0 + j) * STEP;
            uint32_t pk[STEP / 2];
            float corr = 1.f, lsum = 0.f;
            if (sl2 > 0.f) {
                // fast path: maximum on the raw scores, then per pair of elements one packed
                // FMA and either two EX2 or the packed cubic (POLY_PAIRS of every 8 pairs, so
                // that the special-function unit and the FMA pipe share the exponentials)
                const bool diagonal = __any_sync(0xffffffffu, t0 + STEP - 1 > pos);
                float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                if (diagonal) {  // mask
#pragma unroll
                    for (int c = 0; c < STEP; ++c) {
                        float v = __uint_as_float(sr[c >> 5][c & 31]);
                        v = (t0 + c <= pos) ? v : -INFINITY;
                        sr[c >> 5][c & 31] = __float_as_uint(v);
                        m4[c & 3] = fmaxf(m4[c & 3], v);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < STEP; c += 2)
                        m4[(c >> 1) & 3] = max3(m4[(c >> 1) & 3], __uint_as_float(sr[c >> 5][c & 31]),
                                                __uint_as_float(sr[(c + 1) >> 5][(c + 1) & 31]));
                }
                const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * sl2;
                // keep the reference maximum unless it would let a weight exceed 2^8
                if (mx > m_ref + 8.f) {
                    corr = ex2(m_ref - mx);  // 0 on the first step
                    m_ref = mx;
                }
                const float nmu = m_ref == -INFINITY ? 0.f : -m_ref;
                const uint64_t sl2x2 = pack_f32x2(sl2, sl2), nmux2 = pack_f32x2(nmu, nmu);
                uint64_t ls2[4] = {0ull, 0ull, 0ull, 0ull};
                auto weights = [&](auto use_poly) {
#pragma unroll
                    for (int c = 0; c < STEP; c += 2) {
                        const uint64_t y =
                            fma_f32x2(pack_f32x2(__uint_as_float(sr[c >> 5][c & 31]),
                                                 __uint_as_float(sr[(c + 1) >> 5][(c + 1) & 31])),
                                      sl2x2, nmux2);
                        float y0, y1, e0, e1;
                        unpack_f32x2(y, y0, y1);
                        if (decltype(use_poly)::value && ((c >> 1) & 7) < POLY_PAIRS) {
                            exp2_poly_x2(pack_f32x2(fmaxf(y0, -126.f), fmaxf(y1, -126.f)), e0, e1);
                        } else {
                            e0 = ex2(y0);
                            e1 = ex2(y1);
                        }
                        ls2[(c >> 1) & 3] = add_f32x2(ls2[(c >> 1) & 3], pack_f32x2(e0, e1));
                        pk[c >> 1] = pack_bf16x2(e0, e1);
                    }
                };
                // masked elements must come out as exact zeros: the diagonal steps keep EX2
                if (diagonal) weights(std::false_type{}); else weights(std::true_type{});
                float a0, a1, b0, b1;
                unpack_f32x2(add_f32x2(ls2[0], ls2[1]), a0, a1);
                unpack_f32x2(add_f32x2(ls2[2], ls2[3]), b0, b1);
                lsum = (a0 + a1) + (b0 + b1);
            } else {
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < STEP; ++c) {
                    float v = __uint_as_float(sr[c >> 5][c & 31]) * sl2;
                    v = (t0 + c <= pos) ? v : -INFINITY;
                    sr[c >> 5][c & 31] = __float_as_uint(v);
                    mx = fmaxf(mx, v);
                }
                if (mx > m_ref + 8.f) {
                    corr = ex2(m_ref - mx);
                    m_ref = mx;
                }
                const float mu = m_ref == -INFINITY ? 0.f : m_ref;
#pragma unroll
                for (int c = 0; c < STEP; c += 2) {
                    const float e0 = ex2(__uint_as_float(sr[c >> 5][c & 31]) - mu);
                    const float e1 = ex2(__uint_as_float(sr[(c + 1) >> 5][(c + 1) & 31]) - mu);
                    lsum += e0 + e1;
                    pk[c >> 1] = pack_bf16x2(e0, e1);
                }
            }
            l = l * corr + lsum;

            // rescale O (only after the first step, and only once P V of step j-1 is complete)
            if (j >= 1 && __any_sync(0xffffffffu, corr != 1.f)) {
                ok = wait(tb + T_PVDONE + ((j - 1) & 1), ((j - 1) >> 1) & 1);
                if (!ok) break;
                tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < D; c += 32) {
                    uint32_t o[32];
                    tmem_ld32(tcol + lane_base + 2 * STEP + c, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr);
                    tmem_st32(tcol + lane_base + 2 * STEP + c, o);
                }
                tmem_wait_st();
            }
            // P row -> tensor memory, over the scores just read: 64 bf16 in 32 columns
            tmem_st32(tcol + lane_base + (j & 1) * STEP, pk);
            bool zeroed = false;
            // slots past the end of the sequence may hold anything: zero their V rows
            if (ti == 0 && t0 + STEP > L) {  // one warpgroup does it; P V of every tile follows its p_full
                ok = wait(B_VFULL + (j % VS), (j / VS) & 1);
                if (!ok) break;
                const int r0 = max(0, L - t0);                      // first unused row of the step
                const int r1 = min(STEP, ((L + BS - 1) / BS) * BS - t0);  // end of the partial block
                const uint32_t vb = sbase + OFF_V + (j % VS) * TILE_BYTES;
                for (int e = row; e < (r1 - r0) * (D / 8); e += 128) {
                    const int r = r0 + e / (D / 8), c = e % (D / 8);  // 16-byte chunks, 8 per group
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(
                                     vb + (c >> 3) * GROUP_BYTES + r * 128 + (c & 7) * 16),
                                 "r"(0u)
                                 : "memory");
                }
                zeroed = true;
            }
            if (zeroed) fence_proxy_async_smem();
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(tb + T_PFULL + (j & 1)));
        }
        // ---- epilogue: O / l -> bf16 rows, or the unit's partial record when the KV is split ----
        if (ok) ok = wait(tb + T_PVDONE + ((n_steps - 1) & 1), ((n_steps - 1) >> 1) & 1);
        if (n_split > 1) {
            const float2* ml_all = reinterpret_cast<const float2*>(tp.part_ml);
            const float4* o_all = reinterpret_cast<const float4*>(tp.part_o);
            const size_t rec0 = (size_t)group * tp.split_cap * NT + ti;   // record of split s: + s * NT
            if (ok) {
                tc_fence_after_sync();
                const size_t rec = rec0 + (size_t)split * NT;
                if (row_ok)
                    reinterpret_cast<float2*>(tp.part_ml)[rec * 128 + row] =
                        make_float2(m_ref, misc[2] != 0 ? -1.f : l);
                float4* dst = reinterpret_cast<float4*>(tp.part_o) + rec * (D / 4) * 128 + row;
#pragma unroll 1
                for (int c = 0; c < D; c += 64) {  // two tensor-memory loads in flight
                    uint32_t o[2][32];
                    tmem_ld32(tcol + lane_base + 2 * STEP + c, o[0]);
                    tmem_ld32(tcol + lane_base + 2 * STEP + c + 32, o[1]);
                    tmem_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                            for (int i = 0; i < 32; i += 4)
                                dst[(size_t)((c + 32 * hf + i) >> 2) * 128] = make_float4(
                                    __uint_as_float(o[hf][i]), __uint_as_float(o[hf][i + 1]),
                                    __uint_as_float(o[hf][i + 2]), __uint_as_float(o[hf][i + 3]));
                    }
                }
            }
            // The softmax warps of the CTA meet (every one of them gets here: all waits are
            // bounded); one thread counts the unit in, unless some warp gave up.
            asm volatile("bar.sync 1, %0;" ::"r"(NT * 128) : "memory");
            if (warp == 0 && lane == 0) {
                uint32_t last = 0;
                // what the CTA's threads wrote before the barrier is visible to the GPU before
                // the count is (the fence is cumulative over the barrier)
                __threadfence();
                if (misc[1] == 0) {
                    int cur = *reinterpret_cast<volatile int*>(tp.arrive + group), nxt;
                    for (;;) {
                        nxt = ((cur >> 8) == tp.epoch ? cur : (tp.epoch << 8)) + 1;
                        const int prev = atomicCAS(tp.arrive + group, cur, nxt);
                        if (prev == cur) break;
                        cur = prev;
                    }
                    last = (nxt & 255) == n_vis;
                }
                misc[3] = last;
            }
            asm volatile("bar.sync 1, %0;" ::"r"(NT * 128) : "memory");
            if (misc[3] != 0 && n_vis <= 4) {
                merge_few_splits<D, NT>(
                    n_vis, split, m_ref, l, misc[2] != 0, ml_all, o_all, rec0, row, row_ok,
                    p.out + ((size_t)(q0 + qtok) * H + (size_t)kvh * G + hd) * D, tcol, lane_base);
            } else if (misc[3] != 0 && row_ok) {
                // more than four splits: every record from memory, this unit's own included
                __threadfence();
                __nv_bfloat16* dst =
                    p.out + ((size_t)(q0 + qtok) * H + (size_t)kvh * G + hd) * D;
                {
                    float M = -INFINITY;
                    bool bad = false;
                    for (int sp = 0; sp < n_vis; ++sp) {
                        const float2 v = __ldcg(&ml_all[(rec0 + (size_t)sp * NT) * 128 + row]);
                        M = fmaxf(M, v.x);
                        bad |= v.y < 0.f;
                    }
                    float lsum = 0.f;
                    for (int sp = 0; sp < n_vis; ++sp) {
                        const float2 v = __ldcg(&ml_all[(rec0 + (size_t)sp * NT) * 128 + row]);
                        lsum = fmaf(v.x == -INFINITY ? 0.f : ex2(v.x - M), v.y, lsum);
                    }
                    const float inv = (bad || !(lsum > 0.f)) ? 0.f : 1.f / lsum;
#pragma unroll 1
                    for (int c4 = 0; c4 < D / 4; c4 += 8) {
                        float acc[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) acc[i] = 0.f;
                        for (int sp = 0; sp < n_vis; ++sp) {
                            const size_t rec = rec0 + (size_t)sp * NT;
                            const float mx = __ldcg(&ml_all[rec * 128 + row]).x;
                            const float w = mx == -INFINITY ? 0.f : ex2(mx - M) * inv;
                            const float4* src = o_all + (rec * (D / 4) + c4) * 128 + row;
                            float4 x[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) x[i] = __ldcg(src + (size_t)i * 128);
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                acc[4 * i] = fmaf(w, x[i].x, acc[4 * i]);
                                acc[4 * i + 1] = fmaf(w, x[i].y, acc[4 * i + 1]);
                                acc[4 * i + 2] = fmaf(w, x[i].z, acc[4 * i + 2]);
                                acc[4 * i + 3] = fmaf(w, x[i].w, acc[4 * i + 3]);
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            uint4 w4;
                            w4.x = bad ? 0u : pack_bf16x2(acc[i], acc[i + 1]);
                            w4.y = bad ? 0u : pack_bf16x2(acc[i + 2], acc[i + 3]);
                            w4.z = bad ? 0u : pack_bf16x2(acc[i + 4], acc[i + 5]);
                            w4.w = bad ? 0u : pack_bf16x2(acc[i + 6], acc[i + 7]);
                            *reinterpret_cast<uint4*>(dst + c4 * 4 + i) = w4;
                        }
                    }
                }
            }
        } else if (ok) {
            tc_fence_after_sync();
            const bool bad = misc[2] != 0;
            const float inv = bad ? 0.f : 1.f / l;
            __nv_bfloat16* dst =
                p.out + ((size_t)(q0 + qtok) * H + (size_t)kvh * G + hd) * D;
#pragma unroll 1
            for (int c = 0; c < D; c += 32) {
                uint32_t o[32];
                tmem_ld32(tcol + lane_base + 2 * STEP + c, o);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 w;
                        w.x = bad ? 0u : pack_bf16x2(__uint_as_float(o[i]) * inv, __uint_as_float(o[i + 1]) * inv);
                        w.y = bad ? 0u : pack_bf16x2(__uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
                        w.z = bad ? 0u : pack_bf16x2(__uint_as_float(o[i + 4]) * inv, __uint_as_float(o[i + 5]) * inv);
                        w.w = bad ? 0u : pack_bf16x2(__uint_as_float(o[i + 6]) * inv, __uint_as_float(o[i + 7]) * inv);
                        *reinterpret_cast<uint4*>(dst + c + i) = w;
                    }
                }
            }
        }
    }
    // ---- teardown: everyone meets, then the allocating warp returns the tensor memory ----
    tc_fence_before_sync();
    __syncthreads();
    if (warp == C::MMA_WARP) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

// tensor map over the packed queries viewed as [total_q][Hkv][G][D]: box 64 x G x 1 x tokens
// per tile (one 64-dim column group of a row tile per copy)
static int make_q_map(CUtensorMap* map, const void* q, int total_q, int Hkv, int G, int D,
                      int tokens_per_tile) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                 const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                 const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn enc = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            enc = reinterpret_cast<EncodeFn>(ptr);
    });
    if (!enc) {
        set_cuda_error((int)cudaErrorSymbolNotFound);
        return PA_ERR_CUDA;
    }
    cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)G, (cuuint64_t)Hkv, (cuuint64_t)total_q};
    cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)G * D * 2, (cuuint64_t)Hkv * G * D * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)G, 1, (cuuint32_t)tokens_per_tile};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_cuda_error((int)r);
        return PA_ERR_CUDA;
    }
    return PA_OK;
}

template <int D, int NT>
static int launch_prefill_tc(const CUtensorMap& qm, const CUtensorMap& km, const CUtensorMap& vm,
                             const PrefillTcParams& tp, int max_ctas, const DeviceInfo& dev,
                             cudaStream_t st) {
    using C = tc::Cfg<D, NT>;
    static int configured_dev = -1;
    static std::mutex mu;
    {
        std::lock_guard<std::mutex> lk(mu);
        if (configured_dev != dev.device) {
            int rc = check_cuda(cudaFuncSetAttribute(pa_prefill_tc_kernel<D, NT>,
                                                     cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     C::SMEM_BYTES));
            if (rc) return rc;
            configured_dev = dev.device;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(max_ctas);
    cfg.blockDim = dim3(C::THREADS);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return check_cuda(cudaLaunchKernelEx(&cfg, pa_prefill_tc_kernel<D, NT>, qm, km, vm, tp));
}

}  // namespace pk

using namespace pk;

// After the plan come the arrival counters of the row groups (one int per row group and KV
// head; the number of row groups is bounded with one tile per CTA) and the partial records of
// the KV splits: whole 128-row tiles, so a chunk whose sequences end inside a tile, or whose
// head group does not divide 128, holds more rows than it has queries.
static size_t prefill_groups_bound(int64_t total_q, int64_t batch, int G, int Hkv) {
    const int64_t tpt = 128 / G;
    return (size_t)((total_q + tpt - 1) / tpt + batch + 1) * Hkv;
}
static size_t prefill_counter_bytes(int64_t total_q, int64_t batch, int G, int Hkv) {
    return (prefill_groups_bound(total_q, batch, G, Hkv) * sizeof(int) + 255) & ~(size_t)255;
}
// bytes of the records of one split: every bounded row group as one tile of 128 rows, two for
// the last group of each sequence when a CTA takes two tiles
static size_t prefill_split_bytes(int64_t total_q, int64_t batch, int G, int Hkv, int D) {
    const size_t tiles = prefill_groups_bound(total_q, batch, G, Hkv) + (size_t)(batch + 1) * Hkv;
    return tiles * 128 * (size_t)(D + 2) * sizeof(float);
}

static size_t prefill_base_bytes(int64_t batch) {
    const size_t b = PF_WORDS * sizeof(int) + ((size_t)batch + 1) * sizeof(int) + 256;
    return (b + 255) & ~(size_t)255;
}


extern "C" int pa_prefill_workspace_bytes(int32_t max_batch, size_t* bytes) {
    if (!bytes) return PA_ERR_NULL;
    if (max_batch < 0) return PA_ERR_ARG;
    *bytes = prefill_base_bytes(max_batch);
    return PA_OK;
}

extern "C" int pa_prefill_split_workspace_bytes(const pa_shape* shape, int32_t max_batch,
                                                int32_t max_total_q, int32_t max_splits,
                                                size_t* bytes) {
    if (!bytes || !shape) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (max_batch < 0 || max_total_q < 0 || max_splits < 1) return PA_ERR_ARG;
    const int G = shape->num_q_heads / shape->num_kv_heads;
    *bytes = prefill_base_bytes(max_batch) +
             prefill_counter_bytes(max_total_q, max_batch, G, shape->num_kv_heads) +
             (size_t)max_splits *
                 prefill_split_bytes(max_total_q, max_batch, G, shape->num_kv_heads, shape->head_dim);
    return PA_OK;
}

namespace pk {

// Launch shape of the tensor-core path: row tiles per CTA and the KV split length in 64-token
// steps (0 = no split).  Only bounds are known on the host (the chunk's token count, the
// longest context the block table can describe), so this is a cost model, not a plan: rounds
// of CTAs over the SMs times the steps of one unit, a fixed cost per unit, and the traffic of
// the partial records when the KV range is split.
struct TcShape {
    int tiles_per_cta, split_steps, split_cap;
};
// Time of `n_long` units of cost `cl` and `n_short` units of cost `cs` <= cl on `M` SMs when
// the long ones start first and every SM takes the next unit as it becomes free.
static double makespan(int64_t n_long, double cl, int64_t n_short, double cs, int M) {
    const int64_t a = n_long / M, e = n_long % M;
    if (n_short == 0) return (double)(a + (e > 0)) * cl;
    if (e == 0) return a * cl + (double)((n_short + M - 1) / M) * cs;
    // M - e SMs are one long unit behind the others and take short ones until they catch up
    const int64_t k = std::max<int64_t>(1, (int64_t)(cl / cs)), cap = (M - e) * k;
    if (n_short <= cap) return (a + 1) * cl;
    return (a + 1) * cl + (double)((n_short - cap + M - 1) / M) * cs;
}

static TcShape choose_tc_shape(int64_t total_q, int batch, int Hkv, int G, int H, int D,
                               int64_t steps_bound, int sm_count, int64_t cap_fit,
                               int forced_tiles, int forced_split_steps) {
    const int tpt = 128 / G;
    TcShape best = {1, 0, 1};
    double best_t = 1e30;
    for (int nt = 1; nt <= (D == 256 ? 1 : 2); ++nt) {  // head_dim 256: one tile fills the TMEM
        if (forced_tiles && nt != forced_tiles && D != 256) continue;
        const int64_t tpg = (int64_t)nt * tpt;
        // row groups: exact for one sequence; for several, as if they shared the query tokens
        // evenly (a batch of short chunks leaves the second tile of a two-tile CTA empty),
        // never more than the bound the grid is sized with
        const int64_t avg_q = (total_q + batch - 1) / batch;
        const int64_t groups =
            (batch == 1 ? (total_q + tpg - 1) / tpg
                        : std::min<int64_t>(total_q / tpg + batch, batch * ((avg_q + tpg - 1) / tpg))) * Hkv;
        // measured on 512-token chunks at 2K..32K context: microseconds per 64-token step of a
        // CTA, per unit (set-up, pipeline fill, epilogue), and per byte of partial records
        const double step_us = D == 256 ? 1.10 : D == 64 ? (nt == 1 ? 0.66 : 0.88) : (nt == 1 ? 0.65 : 0.84);
        const double unit_us = 8.0;
        auto consider = [&](int64_t T) {
            T = std::min(std::max<int64_t>(T, 1), steps_bound);
            const int64_t S = (steps_bound + T - 1) / T;
            if (S > 1 && (S > cap_fit || (S > 64 && !forced_split_steps))) return;
            if (S > 1 && !forced_split_steps && T < 8) return;  // a unit must be worth its set-up
            const int64_t r = steps_bound - (S - 1) * T;        // steps of the last split
            const bool even = r == T;
            double t = makespan(even ? groups * S : groups * (S - 1), T * step_us + unit_us,
                                even ? 0 : groups, r * step_us + unit_us, sm_count);
            // a split unit writes its record and counts itself in (4.5 us measured); the last
            // one of a row group then reads the other records of its tiles, about 25 us per MB
            // (3.2 us per other split at head_dim 128 with two tiles), half as fast beyond
            // four splits where its loads are not batched
            if (S > 1)
                t += 4.5 + (double)(S - 1) * nt * 128 * D * 4 * (S <= 4 ? 25e-6 : 50e-6);
            if (t < best_t) {
                best_t = t;
                best = {nt, S > 1 ? (int)T : 0, (int)std::max<int64_t>(S, 1)};
            }
        };
        if (forced_split_steps) {
            consider(forced_split_steps);
            continue;
        }
        // even splits, and split lengths in between (a short last split fills SMs that a
        // whole number of equal units would leave idle); a context too short to give every
        // split its 8 steps is looked at once (small calls are bound by the host's issue rate)
        const int64_t s_hi = std::min<int64_t>({cap_fit, 64, steps_bound / 8});
        consider(steps_bound);
        if (s_hi > 1) {
            for (int64_t S = 2; S <= s_hi; ++S) consider((steps_bound + S - 1) / S);
            for (int64_t i = 1; i < 48; ++i) consider(steps_bound * i / 48);
        }
    }
    return best;
}
static thread_local TcShape g_last_shape = {0, 0, 1};

// The number of this call among the calls with a KV split on `workspace` (1 .. 2^23 - 1, then
// from 1 again): the arrival counters carry it, so that what an earlier call left in them
// counts as zero.  `fresh`: the workspace is not in the table (oldest entry replaced first) or
// its numbering starts over -- its counters may hold anything and are cleared.
static int next_epoch(const void* workspace, bool* fresh) {
    struct Entry {
        const void* ws;
        int epoch;
    };
    static std::mutex mu;
    static Entry table[64] = {};
    static int next = 0;
    std::lock_guard<std::mutex> lk(mu);
    for (Entry& e : table)
        if (e.ws == workspace) {
            e.epoch = e.epoch + 1 < (1 << 23) ? e.epoch + 1 : 1;
            *fresh = e.epoch == 1;
            return e.epoch;
        }
    table[next] = Entry{workspace, 1};
    next = (next + 1) % 64;
    *fresh = true;
    return 1;
}

// What pa_prefill_split launches for these arguments (host arithmetic only).  tiles_per_cta 0
// = the warp-level kernel.
static int select_launch(const pa_shape* shape, int batch, int64_t total_q, int max_blocks_per_seq,
                         size_t workspace_bytes, int kv_split_tokens, int sm_count, TcShape* out) {
    const int G = shape->num_q_heads / shape->num_kv_heads, H = shape->num_q_heads, D = shape->head_dim;
    const size_t base_bytes = prefill_base_bytes(batch);
    if (workspace_bytes < base_bytes) return PA_ERR_WORKSPACE;
    // tensor-core path: 128-row tiles of (token, head) pairs of one KV-head group
    static const bool force_mma = [] {
        const char* e = std::getenv("PAGEDKV_PREFILL");
        return e && std::string(e) == "mma";
    }();
    static const int forced_tiles = [] {
        const char* e = std::getenv("PAGEDKV_PREFILL_TILES");
        const int v = e ? std::atoi(e) : 0;
        return v == 1 || v == 2 ? v : 0;
    }();
    *out = TcShape{0, 0, 1};
    if (force_mma) return PA_OK;
    const int64_t steps_bound = std::max<int64_t>(1, ((int64_t)max_blocks_per_seq * BS + 63) / 64);
    const size_t per_split = prefill_split_bytes(total_q, batch, G, shape->num_kv_heads, D);
    const size_t fixed_bytes = base_bytes + prefill_counter_bytes(total_q, batch, G, shape->num_kv_heads);
    const int64_t cap_fit =
        workspace_bytes > fixed_bytes ? (int64_t)((workspace_bytes - fixed_bytes) / per_split) : 0;
    int forced_steps = 0;
    if (kv_split_tokens > 0) {
        forced_steps = (kv_split_tokens + 63) / 64;
        if (forced_steps >= steps_bound) kv_split_tokens = -1;  // one split covers everything
        else if ((steps_bound + forced_steps - 1) / forced_steps > cap_fit) return PA_ERR_WORKSPACE;
    }
    *out = kv_split_tokens < 0
               ? choose_tc_shape(total_q, batch, shape->num_kv_heads, G, H, D, steps_bound, sm_count,
                                 1, forced_tiles, 0)
               : choose_tc_shape(total_q, batch, shape->num_kv_heads, G, H, D, steps_bound, sm_count,
                                 cap_fit, forced_tiles, forced_steps);
    return PA_OK;
}
}  // namespace pk

extern "C" int pa_prefill_select_launch(const pa_shape* shape, int32_t batch, int32_t total_q,
                                        int32_t max_blocks_per_seq, size_t workspace_bytes,
                                        int32_t kv_split_tokens, int32_t sm_count,
                                        int32_t* tiles_per_cta, int32_t* split_tokens,
                                        int32_t* kv_splits) {
    if (!shape || !tiles_per_cta || !split_tokens || !kv_splits) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (batch <= 0 || total_q <= 0 || max_blocks_per_seq < 0 || sm_count <= 0) return PA_ERR_ARG;
    TcShape ts;
    rc = select_launch(shape, batch, total_q, max_blocks_per_seq, workspace_bytes, kv_split_tokens,
                       sm_count, &ts);
    if (rc) return rc;
    *tiles_per_cta = ts.tiles_per_cta;
    *split_tokens = ts.split_steps * 64;
    *kv_splits = ts.split_cap;
    return PA_OK;
}

extern "C" int pa_prefill_last_launch(int32_t* tiles_per_cta, int32_t* kv_split_tokens,
                                      int32_t* kv_splits) {
    if (!tiles_per_cta || !kv_split_tokens || !kv_splits) return PA_ERR_NULL;
    *tiles_per_cta = g_last_shape.tiles_per_cta;
    *kv_split_tokens = g_last_shape.split_steps * 64;
    *kv_splits = g_last_shape.split_cap;
    return PA_OK;
}

extern "C" int pa_prefill_split(const pa_shape* shape, const void* q, const void* k_cache,
                                const void* v_cache, const int32_t* block_tables,
                                int32_t max_blocks_per_seq, const int32_t* ctx_lens,
                                const int32_t* cu_q_lens, int32_t batch, int32_t total_q,
                                float scale, void* out, void* workspace, size_t workspace_bytes,
                                int32_t kv_split_tokens, int32_t* dev_status, void* cuda_stream) {
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
    if ((int64_t)total_q * shape->num_q_heads / 8 >= INT32_MAX) return PA_ERR_ARG;  // rows of the merge grid
    const size_t base_bytes = prefill_base_bytes(batch);
    if (workspace_bytes < base_bytes) return PA_ERR_WORKSPACE;
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
    const int H = shape->num_q_heads, D = shape->head_dim;

    PrefillPlanParams plan;
    plan.ctx_lens = ctx_lens;
    plan.cu_q_lens = cu_q_lens;
    plan.batch = batch;
    plan.max_blocks = max_blocks_per_seq;
    plan.total_q = total_q;
    TcShape ts = {0, 0, 1};
    rc = select_launch(shape, batch, total_q, max_blocks_per_seq, workspace_bytes, kv_split_tokens,
                       dev.sm_count, &ts);
    if (rc) return rc;
    const bool use_tc = ts.tiles_per_cta != 0;
    g_last_shape = use_tc ? ts : TcShape{0, 0, 1};
    plan.tpg = use_tc ? ts.tiles_per_cta * (128 / G) : 16 / G;  // 128 / G rounds down
    plan.split_steps = ts.split_steps;
    plan.hdr = hdr;
    plan.gstart = hdr + PF_WORDS;
    plan.status = dev_status ? dev_status : hdr + PF_STATUS;
    const bool fold_plan = use_tc && batch <= 32;  // the attention CTAs plan for themselves
    if (!fold_plan) {
        // launched as a programmatic dependent of whatever precedes it in the stream (the
        // previous chunk's merge): its launch latency hides under that kernel's tail
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1);
        cfg.blockDim = dim3(1024);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        count_launch();
        rc = check_cuda(cudaLaunchKernelEx(&cfg, pa_prefill_plan_kernel, plan));
        if (rc) return rc;
    }

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
    pp.H = H;
    pp.Hkv = shape->num_kv_heads;
    pp.G = G;
    pp.NB = shape->num_blocks;
    pp.tpg = plan.tpg;
    pp.scale_log2 = scale * 1.4426950408889634f;
    if (use_tc) {
        CUtensorMap qm;
        rc = make_q_map(&qm, q, total_q, pp.Hkv, G, D, 128 / G);
        if (rc) return rc;
        PrefillTcParams tp;
        tp.base = pp;
        tp.tokens_per_tile = 128 / G;
        tp.split_steps = ts.split_steps;
        tp.split_cap = ts.split_cap;
        tp.fold_plan = fold_plan ? 1 : 0;
        tp.total_q = total_q;
        // counters, then the (exponent, sum) pairs of every record, then the rows
        uint8_t* after_plan = static_cast<uint8_t*>(workspace) + base_bytes;
        const size_t n_rec = (size_t)((total_q / plan.tpg + batch + 1) * pp.Hkv) * ts.split_cap *
                             ts.tiles_per_cta;
        tp.arrive = reinterpret_cast<int*>(after_plan);
        tp.part_ml = reinterpret_cast<float*>(after_plan + prefill_counter_bytes(total_q, batch, G, pp.Hkv));
        tp.part_o = tp.part_ml + n_rec * 128 * 2;
        tp.epoch = 0;
        if (ts.split_steps) {
            bool fresh = false;
            tp.epoch = next_epoch(workspace, &fresh);
            if (fresh) {  // never seen (or long ago): no word may look like a count of this epoch
                rc = check_cuda(cudaMemsetAsync(
                    after_plan, 0, prefill_counter_bytes(total_q, batch, G, pp.Hkv), st));
                if (rc) return rc;
            }
        }
        const int64_t max_ctas = ((int64_t)total_q / plan.tpg + batch) * pp.Hkv * ts.split_cap;
        if (max_ctas > INT32_MAX) return PA_ERR_ARG;
        const bool two = ts.tiles_per_cta == 2;
        return D == 256  ? launch_prefill_tc<256, 1>(qm, km, vm, tp, (int)max_ctas, dev, st)
               : D == 128 ? (two ? launch_prefill_tc<128, 2>(qm, km, vm, tp, (int)max_ctas, dev, st)
                                 : launch_prefill_tc<128, 1>(qm, km, vm, tp, (int)max_ctas, dev, st))
                          : (two ? launch_prefill_tc<64, 2>(qm, km, vm, tp, (int)max_ctas, dev, st)
                                 : launch_prefill_tc<64, 1>(qm, km, vm, tp, (int)max_ctas, dev, st));
    }
    return D == 256   ? launch_prefill<256>(km, vm, pp, dev, st)
           : D == 128 ? launch_prefill<128>(km, vm, pp, dev, st)
                      : launch_prefill<64>(km, vm, pp, dev, st);
}

extern "C" int pa_prefill(const pa_shape* shape, const void* q, const void* k_cache,
                          const void* v_cache, const int32_t* block_tables,
                          int32_t max_blocks_per_seq, const int32_t* ctx_lens,
                          const int32_t* cu_q_lens, int32_t batch, int32_t total_q, float scale,
                          void* out, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                          void* cuda_stream) {
    return pa_prefill_split(shape, q, k_cache, v_cache, block_tables, max_blocks_per_seq, ctx_lens,
                            cu_q_lens, batch, total_q, scale, out, workspace, workspace_bytes, 0,
                            dev_status, cuda_stream);
}
