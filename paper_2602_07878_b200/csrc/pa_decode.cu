// Paged-attention decode for sm_100a: plan -> partition attention -> combine.
//
// Partition attention is organised around independent warps.  A warp owns a private ring
// of shared-memory slots; one slot holds the K tile and the V tile (16 tokens x D) of one
// KV block of one KV head, fetched by TMA (128-byte swizzle) and announced by an
// mbarrier.  The warp walks the block table itself, keeps NSLOT-1 blocks in flight across
// unit boundaries, and computes  S = Q K^T  and  O += P V  with warp-level bf16 MMAs whose
// M dimension carries the query heads of the KV head's group.  A unit of work is
// (sequence, KV head, partition of at most 512 tokens); units are handed out longest
// first from a device-built list through an atomic counter, so a 32K-token sequence
// becomes 64+ units that spread over the whole chip next to the short ones.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <utility>
#include <vector>

#include "attn_block.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace pk {

// ======================================================================================
// plan kernel (one CTA): validate lengths, pick the partition size, list the work items
// ======================================================================================
constexpr int PLAN_THREADS = 256;   // small enough to sit beside the previous call's combine CTAs
constexpr int PLAN_WARPS = PLAN_THREADS / 32;
constexpr int SEQ_CACHE = 1024;     // sequences whose (length, first partial) stay in shared memory

constexpr int COMBINE_LONG = 32;  // rows with more partitions get a whole CTA in the combine

struct PlanParams {
    const int32_t* seq_lens;
    int batch;
    int max_blocks;
    int Hkv;
    int H;              // query heads (rows per item that a split sequence sends to the combine)
    int forced_p;       // 0 = automatic
    int no_direct;      // 1 = every sequence goes through the combine kernel
    int64_t item_cap;   // records the workspace can hold
    int total_warps;    // decode warps on the chip
    // Of the region this call fills: seq_info holds per sequence (first partial index,
    // partitions); multi lists the sequences whose rows the combine kernel writes, those with
    // more than COMBINE_LONG partitions from the front, those with 0 or 2..COMBINE_LONG from the
    // back; records holds per item (b, tok0, ntok | flags, partial index).
    PlanAddr plan;
    int* status;
};

__device__ __forceinline__ int clamp_len(int L, int max_tok, bool& bad) {
    if (L < 0 || L > max_tok) {
        bad = true;
        return 0;
    }
    return L;
}

// The kernel reads seq_lens and fills the plan region that the previous call on this workspace
// did not use, and only then waits for the kernels before it in the stream: launched behind
// the combine kernel of the previous call, it runs beside it.  (What precedes it in the stream
// and lets its dependents go early must therefore not be what writes seq_lens; no kernel of
// this library does.)
__global__ void __launch_bounds__(PLAN_THREADS) pa_plan_kernel(const PlanParams p) {
    // per warp: items for each candidate size, items of the forced size, then for each candidate
    // the items of sequences that are split (their rows go through the combine) and the tokens
    __shared__ long long red[10][PLAN_WARPS];
    __shared__ int s_P, s_bad;
    __shared__ int hist[MAX_PART / BS + 1], start[MAX_PART / BS + 1], cursor[MAX_PART / BS + 1];
    __shared__ int scan_warp[PLAN_WARPS];
    __shared__ int s_carry, s_multi, s_long;
    __shared__ int2 s_seq[SEQ_CACHE];  // (length, first partial index) of the first sequences

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int max_tok = p.max_blocks * BS;
    const int cand[4] = {64, 128, 256, 512};
    pdl_launch_dependents();  // the attention kernel may set up while the plan is made
    // The switch was last written at the end of an earlier call's plan kernel, and that call's
    // attention kernel has started since: no wait is needed to read it.
    const int gen = p.plan.fixed[HDR_GEN] + 1;
    const PlanView pv = plan_view(p.plan, gen);

    // ---- pass 1: item counts for each candidate partition size ------------------------
    long long cnt[10] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    bool bad = false;
    for (int b = tid; b < p.batch; b += PLAN_THREADS) {
        const int L = clamp_len(p.seq_lens[b], max_tok, bad);
        if (b < SEQ_CACHE) s_seq[b].x = L;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int np = (L + cand[c] - 1) / cand[c];
            cnt[c] += np;
            if (np > 1) cnt[5 + c] += np;
        }
        if (p.forced_p > 0) cnt[4] += (L + p.forced_p - 1) / p.forced_p;
        cnt[9] += L;
    }
#pragma unroll
    for (int c = 0; c < 10; ++c) {
        long long v = cnt[c];
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) red[c][warp] = v;
    }
    if (tid == 0) s_bad = 0, s_multi = 0, s_long = 0;
    if (tid < MAX_PART / BS + 1) hist[tid] = 0, cursor[tid] = 0;
    __syncthreads();
    if (bad) s_bad = 1;
    if (warp == 0) {
        // lane w holds warp w's counts; one shuffle tree per candidate, every lane ends with
        // the totals
        long long tot[10];
#pragma unroll
        for (int c = 0; c < 10; ++c) {
            long long v = lane < PLAN_WARPS ? red[c][lane] : 0;
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            tot[c] = v;
        }
        int P = 0;
        if (p.forced_p > 0) {
            P = tot[4] <= p.item_cap ? p.forced_p : 0;
        } else {
            // The size that minimises an estimate of the step, in KV tokens streamed by one
            // warp: its share of all tokens (or one whole unit, when there are fewer units than
            // warps), half a unit for the uneven end of the dynamic hand-out, and the combine --
            // a partial row is about as many bytes as one token of one KV head, written and read
            // back, at a quarter of the streaming efficiency.  Measured: workload 2 (64 sequences
            // of at most 2048 tokens) is 3 % faster at 256 than at 512, workloads 3 and 5 (long
            // sequences, many partials) 1.5 and 4 % slower.  Never a size whose items do not fit
            // the workspace.
            const float W = (float)p.total_warps;
            const float share = (float)tot[9] * p.Hkv / W;
            float best = 3.4e38f;
            for (int c = 3; c >= 0; --c) {
                if (tot[c] > p.item_cap) break;
                const float Pc = (float)cand[c];
                const float t = fmaxf(share, Pc) + 0.5f * Pc + 8.f * (float)tot[5 + c] * p.H / W;
                if (t < best) best = t, P = cand[c];
            }
        }
        if (lane == 0) {
            s_P = P;
            s_carry = 0;
        }
    }
    __syncthreads();
    const int P = s_P;
    int n_items = 0;
    if (P == 0) {  // plan does not fit: no work, combine writes zero rows
        for (int b = tid; b < p.batch; b += PLAN_THREADS) {
            pv.seq_info[b] = make_int2(0, 0);
            pv.multi[b] = b;
        }
        if (tid == 0) {
            pv.hdr[HDR_N_MULTI] = p.batch;
            pv.hdr[HDR_N_LONG] = 0;
            pv.hdr[HDR_N_ITEMS] = 0;
            pv.hdr[HDR_N_UNITS] = 0;
            pv.hdr[HDR_P] = 0;
            pv.hdr[HDR_COUNTER] = 3 * p.total_warps;
            atomicOr(p.status, PA_STATUS_WORKSPACE | (s_bad ? PA_STATUS_BAD_SEQ_LEN : 0));
        }
    } else {
        // ---- pass 2: exclusive scan of partitions per sequence, histogram of item sizes ----
        const int full_bin = P / BS;
        for (int base = 0; base < p.batch; base += PLAN_THREADS) {
            const int b = base + tid;
            int np = 0;
            if (b < p.batch) {
                bool dummy = false;
                const int L = b < SEQ_CACHE ? s_seq[b].x : clamp_len(p.seq_lens[b], max_tok, dummy);
                np = (L + P - 1) / P;
                // merged (or zeroed) by the combine kernel
                if (np > COMBINE_LONG) pv.multi[atomicAdd(&s_long, 1)] = b;
                else if (np != 1) pv.multi[p.batch - 1 - atomicAdd(&s_multi, 1)] = b;
                if (np > 0) {
                    if (np > 1) atomicAdd(&hist[full_bin], np - 1);
                    const int last = L - (np - 1) * P;
                    atomicAdd(&hist[(last + BS - 1) / BS], 1);
                }
            }
            int incl = np;
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            if (lane == 31) scan_warp[warp] = incl;
            __syncthreads();
            // inclusive over warps, every warp for itself
            int upto = 0, total = 0;
#pragma unroll
            for (int w = 0; w < PLAN_WARPS; ++w) {
                const int v = scan_warp[w];
                if (w < warp) upto += v;
                total += v;
            }
            const int carry = s_carry;
            if (b < p.batch) {
                const int first = carry + upto + incl - np;
                pv.seq_info[b] = make_int2(first, np);
                if (b < SEQ_CACHE) s_seq[b].y = first;
            }
            __syncthreads();
            if (tid == 0) s_carry = carry + total;
        }
        __syncthreads();
        n_items = s_carry;
        if (warp == 0) {  // larger items first: exclusive scan of the histogram from the top bin down
            static_assert(MAX_PART / BS == 32, "one lane per bin");
            const int nb = MAX_PART / BS - lane;
            const int v = hist[nb];
            int incl = v;
            for (int o = 1; o < 32; o <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += u;
            }
            start[nb] = incl - v;
        }
        if (tid == 0) {
            pv.hdr[HDR_N_ITEMS] = n_items;
            pv.hdr[HDR_N_MULTI] = s_multi;
            pv.hdr[HDR_N_LONG] = s_long;
            pv.hdr[HDR_N_UNITS] = n_items * p.Hkv;
            pv.hdr[HDR_P] = P;
            pv.hdr[HDR_COUNTER] = 3 * p.total_warps;
            if (s_bad) atomicOr(p.status, PA_STATUS_BAD_SEQ_LEN);
        }
        __syncthreads();

        // ---- pass 3: the records, larger items first ------------------------------------------
        auto emit = [&](int b, int L, int np, int first, int part) {
            const int tok0 = part * P;
            const int ntok = min(P, L - tok0);
            const int nb = (ntok + BS - 1) / BS;
            const int pos = start[nb] + atomicAdd(&cursor[nb], 1);
            pv.records[pos] =
                make_int4(b, tok0, ntok | (np == 1 && !p.no_direct ? REC_DIRECT : 0), first + part);
        };
        if (p.batch <= SEQ_CACHE) {
            // one thread per item: its sequence is the last one whose first partial index is not
            // above the item (sequences without tokens share theirs with the next one)
            for (int j = tid; j < n_items; j += PLAN_THREADS) {
                int lo = 0, hi = p.batch - 1;
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (s_seq[mid].y <= j) lo = mid;
                    else hi = mid - 1;
                }
                const int2 sq = s_seq[lo];
                emit(lo, sq.x, (sq.x + P - 1) / P, sq.y, j - sq.y);
            }
        } else {
            // one warp per sequence, lanes over its partitions
            for (int b = warp; b < p.batch; b += PLAN_WARPS) {
                bool dummy = false;
                const int L = b < SEQ_CACHE ? s_seq[b].x : clamp_len(p.seq_lens[b], max_tok, dummy);
                const int np = (L + P - 1) / P;
                if (np == 0) continue;
                const int first = b < SEQ_CACHE ? s_seq[b].y : pv.seq_info[b].x;
                for (int part = lane; part < np; part += 32) emit(b, L, np, first, part);
            }
        }
    }
    // Everything above went to a region that no kernel in flight reads.  This grid must not
    // complete before the kernels of the previous call have (the attention kernel behind it
    // waits for this grid only), and the switch must not move while they may still read it.
    pdl_wait();
    if (tid == 0) {
        p.plan.fixed[HDR_GEN] = gen;
        p.plan.fixed[HDR_N_ITEMS] = n_items;
        p.plan.fixed[HDR_P] = P;
    }
}

// ======================================================================================
// partition attention
// ======================================================================================
struct DecodeParams {
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    const int32_t* block_tables;
    PlanAddr plan;
    float* partial_o;    // [item][H][D]  un-normalised
    float2* partial_ml;  // [item][H]     (running max in log2 units, row sum)
    int* status;
    int max_blocks, H, Hkv, G, NB;
    float scale_log2;
    // elements between the [H, D] rows of consecutive sequences in q and in out (H * D when
    // they are contiguous; larger when they are views into wider tensors)
    int64_t q_stride, out_stride;
};


template <int D, bool HI>
struct UnitRegs {
    int b, tok0, ntok, pidx, kvh;
    int nblk;
    bool direct, valid, bad;
    int id;                                  // this lane's block id (block index = lane)
    uint32_t qa[D / 16][HI ? 4 : 2];         // A fragments of Q for every k-step
    // q in host memory: the group's rows as fetched, 16 bytes per lane and piece (piece
    // i * 32 + lane of the 8 x D block), turned into fragments when the unit becomes current
    uint4 qraw[D / 32];
};

// QH: q lives in pinned host memory (pa_decode_host).  Four-byte fragment loads would cross the
// host link as 16-byte reads; the warp instead fetches the rows of a unit's head group with
// 16-byte loads per lane (512 contiguous bytes per instruction), one unit ahead like the block
// ids, and sorts them into fragments through a small shared-memory buffer.  At most 8 heads per
// group and head_dim 64 or 128.
template <int D, bool HI, int NW, int NSLOT, bool QH = false>
__global__ void __launch_bounds__(NW * 32, 1)
pa_decode_kernel(const __grid_constant__ CUtensorMap kmap,
                 const __grid_constant__ CUtensorMap vmap, const DecodeParams p) {
    constexpr int HALVES = D / 64;         // 128-byte swizzled column groups per row
    constexpr int HALF_BYTES = BS * 128;   // 2 KiB: 16 tokens x 64 dims
    constexpr int TILE = HALVES * HALF_BYTES;
    constexpr int SLOT = 2 * TILE;         // K tile then V tile
    constexpr int KS = D / 16;
    constexpr int NT = D / 8;
    constexpr int QW = HI ? 4 : 2;
    using Unit = UnitRegs<D, HI>;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t slots = base + warp * (NSLOT * SLOT);
    const uint32_t bars = base + NW * NSLOT * SLOT + warp * (NSLOT * 8);
    // Head_dim 256: the output accumulator alone takes 128 registers per thread, so the Q
    // fragments of the next unit are parked in shared memory (one word per lane and fragment)
    // instead of in a second set of registers, and fetched when that unit becomes current.
    constexpr bool QSTASH = D == 256;
    const uint32_t stash = base + NW * NSLOT * SLOT + NW * NSLOT * 8 + warp * (KS * QW * 128) + lane * 4;
    static_assert(!QH || (!HI && D <= 128), "host q: groups of at most 8 heads, head_dim 64 or 128");
    const uint32_t qrows = base + NW * NSLOT * SLOT + NW * NSLOT * 8 + warp * (8 * D * 2);  // QH only

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < NSLOT; ++s) mbar_init(bars + 8 * s, 1);
        mbar_init_fence();
        tma_prefetch_desc(&kmap);
        tma_prefetch_desc(&vmap);
    }
    __syncwarp();
    pdl_wait();               // the plan (and everything before it) is complete and visible
    // Only now may the combine CTAs take their seats: they start once every CTA of this grid
    // has passed this point, i.e. after the plan grid has completed, so the plan's lists are
    // theirs to read even before they wait for this grid's partial results.
    pdl_launch_dependents();

    const PlanView pv = plan_view(p.plan, p.plan.fixed[HDR_GEN]);
    const int n_units = pv.hdr[HDR_N_UNITS];
    const int total_warps = NW * gridDim.x;
    const int gw = warp * gridDim.x + blockIdx.x;
    const int G = p.G, H = p.H, Hkv = p.Hkv;
    const uint32_t* q32 = reinterpret_cast<const uint32_t*>(p.q);

    // ---- unit fetch pipeline: work id -> record -> (block ids, Q fragments) ------------
    auto load_record = [&](int w, int4& rec, int& kvh, bool& valid) {
        valid = w < n_units;
        rec = make_int4(0, 0, 0, 0);
        kvh = 0;
        if (valid) {
            const int item = w / Hkv;
            kvh = w - item * Hkv;
            rec = __ldg(&pv.records[item]);
        }
    };
    auto st_stash = [&](int ks, int i, uint32_t v) {
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(stash + (ks * QW + i) * 128), "r"(v) : "memory");
    };
    // `parked`: the fragments go to the stash (head_dim 256, the unit after the current one)
    auto build = [&](const int4& rec, int kvh, bool valid, Unit& u, bool parked) {
        u.valid = valid;
        u.b = rec.x;
        u.tok0 = rec.y;
        u.ntok = rec.z & 0xFFFF;
        u.direct = (rec.z & REC_DIRECT) != 0;
        u.pidx = rec.w;
        u.kvh = kvh;
        u.nblk = (u.ntok + BS - 1) / BS;
        u.bad = false;
        u.id = 0;
        if (valid && lane < u.nblk)
            u.id = __ldg(&p.block_tables[(size_t)u.b * p.max_blocks + u.tok0 / BS + lane]);
        const size_t row0 = valid ? (size_t)u.b * p.q_stride + (size_t)kvh * G * D : 0;
        if constexpr (QH) {
            const uint4* q128 = reinterpret_cast<const uint4*>(p.q + row0);
#pragma unroll
            for (int i = 0; i < D / 32; ++i) {
                const int piece = i * 32 + lane;           // 16-byte pieces of the 8 x D block
                u.qraw[i] = valid && piece / (D / 8) < G ? __ldg(&q128[piece])
                                                          : make_uint4(0u, 0u, 0u, 0u);
            }
        } else {
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            // a0: (row g, k 2t..), a2: (row g, k 8+2t..); a1/a3 the same for row g+8
            const size_t c = ks * 16 + 2 * t;
            uint32_t w[QW];
            w[0] = valid && g < G ? __ldg(&q32[(row0 + (size_t)g * D + c) >> 1]) : 0u;
            w[QW == 4 ? 2 : 1] = valid && g < G ? __ldg(&q32[(row0 + (size_t)g * D + c + 8) >> 1]) : 0u;
            if (HI) {
                w[1] = valid && g + 8 < G ? __ldg(&q32[(row0 + (size_t)(g + 8) * D + c) >> 1]) : 0u;
                w[QW - 1] =
                    valid && g + 8 < G ? __ldg(&q32[(row0 + (size_t)(g + 8) * D + c + 8) >> 1]) : 0u;
            }
#pragma unroll
            for (int i = 0; i < QW; ++i) {
                if (QSTASH && parked) st_stash(ks, i, w[i]);
                else u.qa[ks][i] = w[i];
            }
        }
        }
    };
    auto unpark = [&](Unit& u) {  // the parked fragments of the unit that has become current
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int i = 0; i < QW; ++i)
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(u.qa[ks][i]) : "r"(stash + (ks * QW + i) * 128));
    };

    auto unpark_host = [&](Unit& u) {  // QH: the rows fetched for this unit -> A fragments
#pragma unroll
        for (int i = 0; i < D / 32; ++i)
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(qrows + (i * 32 + lane) * 16),
                         "r"(u.qraw[i].x), "r"(u.qraw[i].y), "r"(u.qraw[i].z), "r"(u.qraw[i].w)
                         : "memory");
        __syncwarp();
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const uint32_t a = qrows + (g * D + ks * 16 + 2 * t) * 2;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(u.qa[ks][0]) : "r"(a));
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(u.qa[ks][QW - 1]) : "r"(a + 16));
        }
        __syncwarp();
    };

    Unit U0, U1;
    int4 recB;
    int kvhB;
    bool validB;
    int wraw = 0;  // lane 0: work id of the unit after recB
    {
        int4 r0, r1;
        int k0, k1;
        bool v0, v1;
        load_record(gw, r0, k0, v0);
        load_record(gw + total_warps, r1, k1, v1);
        load_record(gw + 2 * total_warps, recB, kvhB, validB);
        if (lane == 0) wraw = atomicAdd(&pv.hdr[HDR_COUNTER], 1);
        build(r0, k0, v0, U0, false);
        if (QH) unpark_host(U0);
        build(r1, k1, v1, U1, true);
    }

    // groups of at most 8 heads at head_dim 256 take the operand-exchanged form: half the MMAs
    // and half the accumulator registers, where a scheduler holds a single warp
    constexpr bool TR = !HI && !QH && D == 256;
    std::conditional_t<TR, AttnFragT<D, true>, AttnFrag<D, HI, true>> A;
    A.init_lane(lane);
    A.reset();

    uint32_t n_issued = 0, n_done = 0;
    int iu = 0, ib = 0, cb = 0;  // issue cursor (unit 0/1, block), compute cursor
    const float sl2 = p.scale_log2;

    while (U0.valid) {
        // ---- keep the ring full: blocks of U0, then of U1 ---------------------------------
        while (n_issued - n_done < (uint32_t)NSLOT) {
            if (iu == 0 && ib == U0.nblk) iu = 1, ib = 0;
            if (iu == 1 && (!U1.valid || ib == U1.nblk)) break;
            const int id = __shfl_sync(0xffffffffu, iu ? U1.id : U0.id, ib);
            const int kvh = iu ? U1.kvh : U0.kvh;
            if ((unsigned)id >= (unsigned)p.NB) {
                if (iu) U1.bad = true; else U0.bad = true;
                if (lane == 0) atomicOr(p.status, PA_STATUS_BAD_BLOCK_ID);
            }
            if (lane == 0) {
                const uint32_t s = n_issued % NSLOT;
                const uint32_t bar = bars + 8 * s;
                const uint32_t dst = slots + s * SLOT;
                mbar_arrive_expect_tx(bar, SLOT);
                // an id outside the pool is out of the tensor's bounds: TMA fills zeros
#pragma unroll
                for (int hf = 0; hf < HALVES; ++hf) {
                    tma_load_4d(dst + hf * HALF_BYTES, &kmap, bar, hf * 64, 0, kvh, id);
                    tma_load_4d(dst + TILE + hf * HALF_BYTES, &vmap, bar, hf * 64, 0, kvh, id);
                }
            }
            ++n_issued;
            ++ib;
        }

        // ---- one block of U0 -----------------------------------------------------------------
        {
            const uint32_t s = n_done % NSLOT;
            if (!mbar_wait_bounded(bars + 8 * s, (n_done / NSLOT) & 1, WAIT_LIMIT_NS)) {
                if (lane == 0) atomicOr(p.status, PA_STATUS_TIMEOUT);
                // give the copies still in flight a bounded chance to land, then leave
                for (uint32_t c = n_done + 1; c < n_issued; ++c)
                    mbar_wait_bounded(bars + 8 * (c % NSLOT), (c / NSLOT) & 1, WAIT_LIMIT_NS);
                return;
            }
            const uint32_t kbase = slots + s * SLOT, vbase = kbase + TILE;
            const int nvalid = min(BS, U0.ntok - cb * BS);

            A.attend(kbase, vbase, U0.qa, nvalid, nvalid, nvalid, sl2, lane);
            ++n_done;
            ++cb;
        }

        // ---- unit finished: write its result, move to the next unit -----------------------------
        if (cb == U0.nblk) {
            A.reduce_row_sums();
            if constexpr (TR) {
                // this thread: heads 2t and 2t + 1 of the group, dims 16 jj + g and + 8
                const int hA = U0.kvh * G + 2 * t;
                const bool okA = 2 * t < G, okB = 2 * t + 1 < G;
                if (U0.direct) {
                    // neighbours in g exchange a value, so that each stores two dims of one head
                    const float iA = U0.bad ? 0.f : 1.f / A.l0, iB = U0.bad ? 0.f : 1.f / A.l1;
                    const bool even = (g & 1) == 0;
                    const bool ok = even ? okA : okB;
                    uint32_t* dst = reinterpret_cast<uint32_t*>(
                        p.out + (size_t)U0.b * p.out_stride + (size_t)(hA + (even ? 0 : 1)) * D);
#pragma unroll
                    for (int jj = 0; jj < D / 16; ++jj) {
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {
                            const float xA = A.o[jj][2 * hf] * iA, xB = A.o[jj][2 * hf + 1] * iB;
                            const float got = __shfl_xor_sync(0xffffffffu, even ? xB : xA, 4);
                            const uint32_t w = even ? pack_bf16x2(xA, got) : pack_bf16x2(got, xB);
                            if (ok) dst[(16 * jj + 8 * hf + (g & ~1)) >> 1] = w;
                        }
                    }
                } else {
                    const float nanv = __int_as_float(0x7fc00000);
                    const size_t rowA = (size_t)U0.pidx * H + hA;
                    float* dA = p.partial_o + rowA * D;
                    float* dB = dA + D;
#pragma unroll
                    for (int jj = 0; jj < D / 16; ++jj) {
                        if (okA) dA[16 * jj + g] = A.o[jj][0], dA[16 * jj + g + 8] = A.o[jj][2];
                        if (okB) dB[16 * jj + g] = A.o[jj][1], dB[16 * jj + g + 8] = A.o[jj][3];
                    }
                    if (g == 0) {
                        if (okA) p.partial_ml[rowA] = make_float2(U0.bad ? nanv : A.m0, A.l0);
                        if (okB) p.partial_ml[rowA + 1] = make_float2(U0.bad ? nanv : A.m1, A.l1);
                    }
                }
            } else {
                const float l0 = A.l0, l1 = A.l1, m0 = A.m0, m1 = A.m1;
                auto& o = A.o;
                const int h0 = U0.kvh * G + g;
                if (QH && U0.direct) {
                    // host-resident tensors: the rows go out as whole 16-byte pieces per lane (512
                    // contiguous bytes per instruction) instead of 4-byte fragments
                    const float i0 = U0.bad ? 0.f : 1.f / l0;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(qrows + (g * D + nt * 8 + 2 * t) * 2),
                                     "r"(U0.bad ? 0u : pack_bf16x2(o[nt][0] * i0, o[nt][1] * i0))
                                     : "memory");
                    __syncwarp();
                    uint4* orow = reinterpret_cast<uint4*>(p.out + (size_t)U0.b * p.out_stride +
                                                           (size_t)U0.kvh * G * D);
#pragma unroll
                    for (int i = 0; i < D / 32; ++i) {
                        const int piece = i * 32 + lane;
                        if (piece / (D / 8) < G) {
                            uint4 w;
                            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                                         : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w)
                                         : "r"(qrows + piece * 16));
                            orow[piece] = w;
                        }
                    }
                    __syncwarp();
                } else if (U0.direct) {
                    const float i0 = U0.bad ? 0.f : 1.f / l0, i1 = U0.bad ? 0.f : 1.f / l1;
                    if (g < G) {
                        uint32_t* dst = reinterpret_cast<uint32_t*>(
                            p.out + (size_t)U0.b * p.out_stride + (size_t)h0 * D);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
                            dst[nt * 4 + t] = U0.bad ? 0u : pack_bf16x2(o[nt][0] * i0, o[nt][1] * i0);
                    }
                    if (HI && g + 8 < G) {
                        uint32_t* dst = reinterpret_cast<uint32_t*>(
                            p.out + (size_t)U0.b * p.out_stride + (size_t)(h0 + 8) * D);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
                            dst[nt * 4 + t] = U0.bad ? 0u : pack_bf16x2(o[nt][2] * i1, o[nt][3] * i1);
                    }
                } else {
                    const float nanv = __int_as_float(0x7fc00000);
                    if (g < G) {
                        const size_t row = (size_t)U0.pidx * H + h0;
                        float2* dst = reinterpret_cast<float2*>(p.partial_o + row * D);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) dst[nt * 4 + t] = make_float2(o[nt][0], o[nt][1]);
                        if (t == 0) p.partial_ml[row] = make_float2(U0.bad ? nanv : m0, l0);
                    }
                    if (HI && g + 8 < G) {
                        const size_t row = (size_t)U0.pidx * H + h0 + 8;
                        float2* dst = reinterpret_cast<float2*>(p.partial_o + row * D);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) dst[nt * 4 + t] = make_float2(o[nt][2], o[nt][3]);
                        if (t == 0) p.partial_ml[row] = make_float2(U0.bad ? nanv : m1, l1);
                    }
                }
            }
            // advance the fetch pipeline
            U0 = U1;
            if (QSTASH) unpark(U0);
            if (QH) unpark_host(U0);
            build(recB, kvhB, validB, U1, true);
            const int w = __shfl_sync(0xffffffffu, wraw, 0);
            load_record(w, recB, kvhB, validB);
            if (lane == 0) wraw = atomicAdd(&pv.hdr[HDR_COUNTER], 1);
            if (iu == 1) iu = 0; else ib = 0;  // the issue cursor stays where it was
            cb = 0;
            A.reset();
        }
    }
}

// ======================================================================================
// combine: one CTA per (sequence, query head)
// ======================================================================================
struct CombineParams {
    PlanAddr plan;     // unused by COMBINE_MERGE
    const float* partial_o;
    const float2* partial_ml;
    __nv_bfloat16* out;
    int rows;  // batch * H
    int H;
    int64_t out_stride;  // elements between the [H, D] output rows of consecutive sequences
    int counter_reset;
    // COMBINE_TO_PARTIAL: one un-normalised fp32 row and its (max, sum) per output row
    float* part_o;
    float2* part_ml;
    // COMBINE_MERGE: the partitions of row r are row r of each of n_parts records
    int n_parts;
    const float* parts[PA_MAX_PARTS];
};

enum { COMBINE_FINAL = 0, COMBINE_TO_PARTIAL = 1, COMBINE_MERGE = 2 };

// One CTA (4 warps) per (sequence, query head) row.  Every warp finds the row maximum, then
// the warps share the partitions (warp w takes w, w+4, ...), eight independent 512-byte row
// loads at a time, and the four partial sums meet in shared memory.
template <int D, int MODE>
__global__ void __launch_bounds__(128) pa_combine_kernel(const __grid_constant__ CombineParams p) {
    constexpr int VPL = D / 32;  // floats per lane
    constexpr int UB = 8;        // rows in flight per warp
    __shared__ float s_acc[4][D];
    __shared__ float s_den[4];
    const int row = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    pdl_wait();  // partial results of the attention kernel are complete and visible
    const int b = row / p.H, h = row - b * p.H;
    int2 info = make_int2(0, p.n_parts);
    if (MODE != COMBINE_MERGE) {
        const PlanView pv = plan_view(p.plan, p.plan.fixed[HDR_GEN]);
        if (row == 0 && threadIdx.x == 0) pv.hdr[HDR_COUNTER] = p.counter_reset;
        info = pv.seq_info[b];
    }
    if (MODE == COMBINE_FINAL && info.y == 1) return;  // written directly by the attention kernel
    __nv_bfloat16* dst = p.out + (size_t)b * p.out_stride + (size_t)h * D;
    if (info.y == 0) {  // no tokens: a row of zeros (as a partial: weight zero)
        if (MODE == COMBINE_TO_PARTIAL) {
            if (threadIdx.x < D / 2)
                reinterpret_cast<float2*>(p.part_o + (size_t)row * D)[threadIdx.x] =
                    make_float2(0.f, 0.f);
            if (threadIdx.x == 0) p.part_ml[row] = make_float2(-INFINITY, 0.f);
        } else if (threadIdx.x < D / 2) {
            reinterpret_cast<uint32_t*>(dst)[threadIdx.x] = 0u;
        }
        return;
    }
    const int np = info.y, first = info.x;
    // partition i of this row: its (max, sum) pair and its accumulator row
    auto ml_of = [&](int i) -> float2 {
        if (MODE == COMBINE_MERGE)
            return reinterpret_cast<const float2*>(p.parts[i] + (size_t)p.rows * D)[row];
        return p.partial_ml[(size_t)(first + i) * p.H + h];
    };
    auto o_of = [&](int i) -> const float* {
        if (MODE == COMBINE_MERGE) return p.parts[i] + (size_t)row * D;
        return p.partial_o + ((size_t)(first + i) * p.H + h) * D;
    };
    float M = -INFINITY;
    bool bad = false;
    for (int i = lane; i < np; i += 32) {
        const float m = ml_of(i).x;
        bad |= m != m;  // NaN marks a partition that met a bad block id
        M = fmaxf(M, m);
    }
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    bad = __any_sync(0xffffffffu, bad);
    if (M == -INFINITY) M = 0.f;

    float acc[VPL];
#pragma unroll
    for (int i = 0; i < VPL; ++i) acc[i] = 0.f;
    float den = 0.f;
    for (int i0 = warp; i0 < np; i0 += 4 * UB) {
        float2 ml[UB];
        float v[UB][VPL];
#pragma unroll
        for (int u = 0; u < UB; ++u) {
            const int idx = min(i0 + 4 * u, np - 1);
            ml[u] = ml_of(idx);
            const float* src = o_of(idx) + lane * VPL;
            if (VPL >= 4) {
#pragma unroll
                for (int i = 0; i + 3 < VPL; i += 4) {
                    const float4 x = *reinterpret_cast<const float4*>(src + i);
                    v[u][i] = x.x, v[u][i + 1] = x.y, v[u][i + 2] = x.z, v[u][i + 3] = x.w;
                }
            } else {
                const float2 x = *reinterpret_cast<const float2*>(src);
                v[u][0] = x.x, v[u][1] = x.y;
            }
        }
#pragma unroll
        for (int u = 0; u < UB; ++u)
            if (i0 + 4 * u < np) {
                const float w = ex2(ml[u].x - M);
                den += w * ml[u].y;
#pragma unroll
                for (int i = 0; i < VPL; ++i) acc[i] += w * v[u][i];
            }
    }
#pragma unroll
    for (int i = 0; i < VPL; ++i) s_acc[warp][lane * VPL + i] = acc[i];
    if (lane == 0) s_den[warp] = den;
    __syncthreads();
    if (warp != 0) return;
    den = (s_den[0] + s_den[1]) + (s_den[2] + s_den[3]);
    // a row without any token in every part (den == 0) is a row of zeros
    const float inv = MODE == COMBINE_TO_PARTIAL ? 1.f : (bad || den == 0.f) ? 0.f : 1.f / den;
    float o[VPL];
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
        const int c = lane * VPL + i;
        o[i] = ((s_acc[0][c] + s_acc[1][c]) + (s_acc[2][c] + s_acc[3][c])) * inv;
    }
    if (MODE == COMBINE_TO_PARTIAL) {
        float* po = p.part_o + (size_t)row * D + lane * VPL;
#pragma unroll
        for (int i = 0; i < VPL; i += 2)
            *reinterpret_cast<float2*>(po + i) = make_float2(o[i], o[i + 1]);
        if (lane == 0)
            p.part_ml[row] = make_float2(bad ? __int_as_float(0x7fc00000) : M, den);
        return;
    }
    if (VPL >= 4) {
#pragma unroll
        for (int i = 0; i + 3 < VPL; i += 4) {
            uint2 x;
            x.x = bad ? 0u : pack_bf16x2(o[i], o[i + 1]);
            x.y = bad ? 0u : pack_bf16x2(o[i + 2], o[i + 3]);
            *reinterpret_cast<uint2*>(dst + lane * VPL + i) = x;
        }
    } else {
        *reinterpret_cast<uint32_t*>(dst + lane * VPL) = bad ? 0u : pack_bf16x2(o[0], o[1]);
    }
}

// ======================================================================================
// host side
// ======================================================================================
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) ==
                cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

// tensor map over one layer's cache: dims (dim, slot, kv head, block), box 64 x 16 x 1 x 1
int make_cache_map(CUtensorMap* map, const void* base, const pa_shape* s) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) {
        set_cuda_error((int)cudaErrorSymbolNotFound);
        return PA_ERR_CUDA;
    }
    cuuint64_t dims[4] = {(cuuint64_t)s->head_dim, (cuuint64_t)s->block_size,
                          (cuuint64_t)s->num_kv_heads, (cuuint64_t)s->num_blocks};
    cuuint64_t strides[3] = {(cuuint64_t)s->stride_tok * 2, (cuuint64_t)s->stride_head * 2,
                             (cuuint64_t)s->stride_block * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)BS, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims,
                     strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_cuda_error((int)r);
        return PA_ERR_CUDA;
    }
    return PA_OK;
}

WsLayout ws_layout(int H, int D, int64_t batch, int64_t item_cap, size_t bytes) {
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    WsLayout w;
    w.off_region = up(HDR_WORDS * sizeof(int));
    w.off_seqinfo = up(HDR_WORDS * sizeof(int));
    w.off_multi = w.off_seqinfo + up((size_t)batch * sizeof(int2));
    w.off_records = w.off_multi + up((size_t)batch * sizeof(int));
    // an item: its record in either plan region, its (max, sum) pairs and accumulator rows
    const size_t per_item =
        2 * sizeof(int4) + (size_t)H * sizeof(float2) + (size_t)H * D * sizeof(float);
    if (bytes > 0) {
        const size_t fixed = w.off_region + 2 * w.off_records + 4 * 256;
        item_cap = bytes > fixed ? (int64_t)((bytes - fixed) / per_item) : 0;
    }
    w.item_cap = item_cap;
    w.region_bytes = w.off_records + up((size_t)item_cap * sizeof(int4));
    w.off_ml = w.off_region + 2 * w.region_bytes;
    w.off_o = w.off_ml + up((size_t)item_cap * H * sizeof(float2));
    w.total = w.off_o + up((size_t)item_cap * H * D * sizeof(float));
    return w;
}

// Launch with programmatic stream serialization: the kernel may start before the previous
// kernel in the stream has finished and synchronises on it with griddepcontrol.wait.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

struct Variant {
    int nw, nslot;
};

template <int D, bool HI, int NW, int NSLOT, bool QH = false>
static int launch_decode(const CUtensorMap& km, const CUtensorMap& vm, const DecodeParams& dp,
                         const DeviceInfo& dev, int* grid_out, bool launch, cudaStream_t st) {
    auto kern = pa_decode_kernel<D, HI, NW, NSLOT, QH>;
    // at head_dim 256 the Q fragments of the unit after the current one wait in shared memory;
    // with q in host memory a warp sorts the fetched rows of a head group through 8 x D bf16
    const int stash = D == 256 ? NW * (D / 16) * (HI ? 4 : 2) * 32 * 4 : QH ? NW * 8 * D * 2 : 0;
    const int smem = NW * NSLOT * (2 * BS * D * 2) + NW * NSLOT * 8 + stash + 1024;
    if (smem > dev.smem_optin) return PA_ERR_SHAPE;
    static int configured_dev = -1, ctas_per_sm = 0;
    static std::mutex mu;
    {
        std::lock_guard<std::mutex> lk(mu);
        if (configured_dev != dev.device) {
            int rc = check_cuda(cudaFuncSetAttribute(
                kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            if (rc) return rc;
            rc = check_cuda(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ctas_per_sm, kern,
                                                                          NW * 32, smem));
            if (rc) return rc;
            if (ctas_per_sm < 1) return PA_ERR_SHAPE;
            configured_dev = dev.device;
        }
    }
    const int grid = dev.sm_count * ctas_per_sm;
    *grid_out = grid * NW;  // total warps
    if (!launch) return PA_OK;
    count_launch();
    return check_cuda(launch_pdl(kern, dim3(grid), dim3(NW * 32), smem, st, km, vm, dp));
}

template <int D, bool HI>
static int dispatch_variant(Variant v, const CUtensorMap& km, const CUtensorMap& vm,
                            const DecodeParams& dp, const DeviceInfo& dev, int* warps, bool launch,
                            cudaStream_t st, bool q_on_host) {
    if constexpr (!HI && D <= 128) {
        if (q_on_host)
            return launch_decode<D, HI, 8, D == 64 ? 6 : 3, true>(km, vm, dp, dev, warps, launch, st);
    }
    if constexpr (D == 256) {
        // a slot is 16 KiB: four warps with three slots each fill the shared memory
        return launch_decode<D, HI, 4, 3>(km, vm, dp, dev, warps, launch, st);
    } else {
        constexpr int F = D == 64 ? 2 : 1;  // a D=64 slot is half the size: twice the slots
#define PK_CASE(NW_, NS_) \
    if (v.nw == NW_ && v.nslot == NS_) \
        return launch_decode<D, HI, NW_, NS_ * F>(km, vm, dp, dev, warps, launch, st);
        PK_CASE(8, 3)
        PK_CASE(4, 3)
#undef PK_CASE
        return PA_ERR_ARG;
    }
}

static Variant chosen_variant() {
    static Variant v = [] {
        Variant d{8, 3};
        if (const char* e = std::getenv("PAGEDKV_VARIANT")) {
            int a = 0, b = 0;
            if (std::sscanf(e, "%d,%d", &a, &b) == 2) d = Variant{a, b};
        }
        return d;
    }();
    return v;
}

// q in host memory is read in place for groups of at most 8 heads at head_dim 64 or 128
static bool host_q_supported(const pa_shape* s) {
    return s->num_q_heads / s->num_kv_heads <= 8 && s->head_dim <= 128;
}

static int dispatch_decode(const pa_shape* s, const CUtensorMap& km, const CUtensorMap& vm,
                           const DecodeParams& dp, const DeviceInfo& dev, int* warps, bool launch,
                           cudaStream_t st, bool q_on_host = false) {
    const bool hi = s->num_q_heads / s->num_kv_heads > 8;
    const Variant v = chosen_variant();
    const bool qh = q_on_host && host_q_supported(s);
    if (s->head_dim == 256)
        return hi ? dispatch_variant<256, true>(v, km, vm, dp, dev, warps, launch, st, qh)
                  : dispatch_variant<256, false>(v, km, vm, dp, dev, warps, launch, st, qh);
    if (s->head_dim == 128)
        return hi ? dispatch_variant<128, true>(v, km, vm, dp, dev, warps, launch, st, qh)
                  : dispatch_variant<128, false>(v, km, vm, dp, dev, warps, launch, st, qh);
    return hi ? dispatch_variant<64, true>(v, km, vm, dp, dev, warps, launch, st, qh)
              : dispatch_variant<64, false>(v, km, vm, dp, dev, warps, launch, st, qh);
}

// ---- optional per-kernel timing (CUDA events recorded around each of the three launches) ----
struct ProfCall {
    cudaEvent_t ev[4];
};
static std::mutex g_prof_mu;
static bool g_prof_on = false;
static std::vector<ProfCall> g_prof_calls;
static std::vector<ProfCall> g_prof_free;
constexpr size_t PROF_MAX_CALLS = 1 << 16;

static bool prof_begin_call(ProfCall* out) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    if (!g_prof_on || g_prof_calls.size() >= PROF_MAX_CALLS) return false;
    ProfCall c;
    if (!g_prof_free.empty()) {
        c = g_prof_free.back();
        g_prof_free.pop_back();
    } else {
        for (int i = 0; i < 4; ++i)
            if (cudaEventCreate(&c.ev[i]) != cudaSuccess) return false;
    }
    g_prof_calls.push_back(c);
    *out = c;
    return true;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace pk

using namespace pk;

extern "C" int pa_workspace_bytes(const pa_shape* shape, int32_t max_batch,
                                  int64_t max_total_tokens, int32_t partition_tokens,
                                  size_t* bytes) {
    if (!shape || !bytes) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (max_batch < 0 || max_total_tokens < 0) return PA_ERR_ARG;
    if (partition_tokens != 0 &&
        (partition_tokens < BS || partition_tokens > MAX_PART || partition_tokens % BS))
        return PA_ERR_ARG;
    const int64_t pw = partition_tokens ? partition_tokens : 256;
    const int64_t cap = max_total_tokens / pw + max_batch + 1;
    WsLayout w = ws_layout(shape->num_q_heads, shape->head_dim, max_batch, cap, 0);
    *bytes = w.total + 4 * 256;
    return PA_OK;
}

// The combine of pa_decode itself, over the sequences the plan listed.  A fixed grid of CTAs of
// eight warps: first the rows of the long sequences (more than COMBINE_LONG partitions), one
// (sequence, head) row per CTA at a time with warp w taking partitions w, w + 8, ... and the
// eight sums meeting in shared memory; then the rows of the short ones (2..COMBINE_LONG
// partitions, or none: a row of zeros), one row per warp, no shared memory, no barrier.  No CTA
// is spent on rows the attention kernel wrote directly.
template <int D>
__global__ void __launch_bounds__(256) pa_combine_rows_kernel(const __grid_constant__ CombineParams p) {
    constexpr int VPL = D / 32;  // floats per lane
    constexpr int UB = 8;        // partition rows in flight per warp
    __shared__ float s_acc[8][D];
    __shared__ float s_den[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_launch_dependents();
    // The plan's lists were complete before this grid could start (the attention kernel lets
    // its dependents go only after it has seen the plan), so the chain header -> list entry ->
    // sequence record of this CTA's first rows is walked while the attention kernel still runs.
    const int batch = p.rows / p.H;
    const PlanView pv = plan_view(p.plan, p.plan.fixed[HDR_GEN]);
    const int n_long = pv.hdr[HDR_N_LONG] * p.H, n_short = pv.hdr[HDR_N_MULTI] * p.H;
    int2 first_long = make_int2(0, 0), first_short = make_int2(0, 0);
    int first_long_b = 0, first_short_b = 0;
    if ((int)blockIdx.x < n_long) {
        first_long_b = __ldg(&pv.multi[blockIdx.x / p.H]);
        first_long = pv.seq_info[first_long_b];
    }
    if ((int)blockIdx.x * 8 + warp < n_short) {
        first_short_b = __ldg(&pv.multi[batch - 1 - (blockIdx.x * 8 + warp) / p.H]);
        first_short = pv.seq_info[first_short_b];
    }
    pdl_wait();  // partial results of the attention kernel are complete and visible
    if (blockIdx.x == 0 && threadIdx.x == 0) pv.hdr[HDR_COUNTER] = p.counter_reset;

    // sum of w_i * (o_i, l_i) over partitions i = start, start + stride, ... < np of one row
    auto gather = [&](int first, int np, int h, int start, int stride, float M, float (&acc)[VPL],
                      float& den) {
        for (int i0 = start; i0 < np; i0 += UB * stride) {
            float2 ml[UB];
            float v[UB][VPL];
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int idx = min(i0 + u * stride, np - 1);
                ml[u] = p.partial_ml[(size_t)(first + idx) * p.H + h];
                const float* src = p.partial_o + ((size_t)(first + idx) * p.H + h) * D + lane * VPL;
                if (VPL >= 4) {
#pragma unroll
                    for (int i = 0; i + 3 < VPL; i += 4) {
                        const float4 x = *reinterpret_cast<const float4*>(src + i);
                        v[u][i] = x.x, v[u][i + 1] = x.y, v[u][i + 2] = x.z, v[u][i + 3] = x.w;
                    }
                } else {
                    const float2 x = *reinterpret_cast<const float2*>(src);
                    v[u][0] = x.x, v[u][1] = x.y;
                }
            }
#pragma unroll
            for (int u = 0; u < UB; ++u)
                if (i0 + u * stride < np) {
                    const float w = ex2(ml[u].x - M);
                    den += w * ml[u].y;
#pragma unroll
                    for (int i = 0; i < VPL; ++i) acc[i] += w * v[u][i];
                }
        }
    };
    // the row maximum (every lane gets it) and whether a partition was flagged (NaN maximum)
    auto row_max = [&](int first, int np, int h, bool& bad) -> float {
        float M = -INFINITY;
        bad = false;
        for (int i = lane; i < np; i += 32) {
            const float m = p.partial_ml[(size_t)(first + i) * p.H + h].x;
            bad |= m != m;
            M = fmaxf(M, m);
        }
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        bad = __any_sync(0xffffffffu, bad);
        return M == -INFINITY ? 0.f : M;
    };
    auto store = [&](__nv_bfloat16* dst, const float (&o)[VPL], bool zero) {
        if (VPL >= 4) {
#pragma unroll
            for (int i = 0; i + 3 < VPL; i += 4) {
                uint2 x;
                x.x = zero ? 0u : pack_bf16x2(o[i], o[i + 1]);
                x.y = zero ? 0u : pack_bf16x2(o[i + 2], o[i + 3]);
                *reinterpret_cast<uint2*>(dst + i) = x;
            }
        } else {
            *reinterpret_cast<uint32_t*>(dst) = zero ? 0u : pack_bf16x2(o[0], o[1]);
        }
    };

    // ---- long rows: one per CTA ----
    for (int task = blockIdx.x; task < n_long; task += gridDim.x) {
        const bool first = task == (int)blockIdx.x;
        const int b = first ? first_long_b : __ldg(&pv.multi[task / p.H]), h = task % p.H;
        const int2 info = first ? first_long : pv.seq_info[b];
        bool bad;
        const float M = row_max(info.x, info.y, h, bad);
        float acc[VPL];
#pragma unroll
        for (int i = 0; i < VPL; ++i) acc[i] = 0.f;
        float den = 0.f;
        gather(info.x, info.y, h, warp, 8, M, acc, den);
#pragma unroll
        for (int i = 0; i < VPL; ++i) s_acc[warp][lane * VPL + i] = acc[i];
        if (lane == 0) s_den[warp] = den;
        __syncthreads();
        if (warp == 0) {
            den = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) den += s_den[w];
            const bool zero = bad || den == 0.f;  // (a flagged row's sums may be NaN)
            const float inv = zero ? 0.f : 1.f / den;
            float o[VPL];
#pragma unroll
            for (int i = 0; i < VPL; ++i) {
                float t = 0.f;
#pragma unroll
                for (int w = 0; w < 8; ++w) t += s_acc[w][lane * VPL + i];
                o[i] = t * inv;
            }
            store(p.out + (size_t)b * p.out_stride + (size_t)h * D + lane * VPL, o, zero);
        }
        __syncthreads();
    }
    // ---- short rows: one per warp ----
    for (int task = blockIdx.x * 8 + warp; task < n_short; task += gridDim.x * 8) {
        const bool first = task == (int)blockIdx.x * 8 + warp;
        const int b = first ? first_short_b : __ldg(&pv.multi[batch - 1 - task / p.H]), h = task % p.H;
        const int2 info = first ? first_short : pv.seq_info[b];
        bool bad;
        const float M = row_max(info.x, info.y, h, bad);
        float acc[VPL];
#pragma unroll
        for (int i = 0; i < VPL; ++i) acc[i] = 0.f;
        float den = 0.f;
        gather(info.x, info.y, h, 0, 1, M, acc, den);
        const bool zero = info.y == 0 || bad || den == 0.f;
        const float inv = zero ? 0.f : 1.f / den;
#pragma unroll
        for (int i = 0; i < VPL; ++i) acc[i] *= inv;
        store(p.out + (size_t)b * p.out_stride + (size_t)h * D + lane * VPL, acc, zero);
    }
}

template <int MODE>
static cudaError_t launch_combine(int D, int grid, cudaStream_t st, const CombineParams& cp) {
    return D == 256   ? launch_pdl(pa_combine_kernel<256, MODE>, dim3(grid), dim3(128), 0, st, cp)
           : D == 128 ? launch_pdl(pa_combine_kernel<128, MODE>, dim3(grid), dim3(128), 0, st, cp)
                      : launch_pdl(pa_combine_kernel<64, MODE>, dim3(grid), dim3(128), 0, st, cp);
}

// CTAs of pa_combine_rows_kernel that one SM holds (asked once per head_dim).
static int combine_rows_per_sm(int D, int* out) {
    static std::mutex mu;
    static int cached[3] = {0, 0, 0};
    const int i = D == 64 ? 0 : D == 128 ? 1 : 2;
    std::lock_guard<std::mutex> lk(mu);
    if (!cached[i]) {
        int n = 0;
        cudaError_t e =
            D == 256   ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pa_combine_rows_kernel<256>, 256, 0)
            : D == 128 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pa_combine_rows_kernel<128>, 256, 0)
                       : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pa_combine_rows_kernel<64>, 256, 0);
        if (e != cudaSuccess) return check_cuda(e);
        cached[i] = n > 0 ? n : 1;
    }
    *out = cached[i];
    return PA_OK;
}

// The three launches of a decode call.  `part` == nullptr: bf16 rows in `out`; otherwise one
// partial record (un-normalised fp32 rows, then their (max, sum) pairs) in `part`.
static int decode_impl(const pa_shape* shape, const void* q, const void* k_cache,
                       const void* v_cache, const int32_t* block_tables,
                       int32_t max_blocks_per_seq, const int32_t* seq_lens, int32_t batch,
                       float scale, void* out, float* part, void* workspace,
                       size_t workspace_bytes, int32_t partition_tokens, int32_t flags,
                       int32_t* dev_status, void* cuda_stream, int64_t q_stride = 0,
                       int64_t out_stride = 0, bool q_on_host = false) {
    if (!shape) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (batch < 0 || max_blocks_per_seq < 0) return PA_ERR_ARG;
    if (partition_tokens != 0 &&
        (partition_tokens < BS || partition_tokens > MAX_PART || partition_tokens % BS))
        return PA_ERR_ARG;
    if (flags & ~PA_FLAG_REUSE_PLAN) return PA_ERR_ARG;
    if (batch == 0) return PA_OK;
    if (!q || !k_cache || !v_cache || !block_tables || !seq_lens || !(part ? (void*)part : out) ||
        !workspace)
        return PA_ERR_NULL;
    if (!aligned16(q) || !aligned16(part ? (void*)part : out) || !aligned16(k_cache) ||
        !aligned16(v_cache) || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return PA_ERR_ALIGN;
    if ((int64_t)max_blocks_per_seq * BS > INT32_MAX) return PA_ERR_ARG;

    const int H = shape->num_q_heads, D = shape->head_dim;
    // 0 = contiguous; otherwise at least one [H, D] row apart and a multiple of 8 elements so
    // that every row stays 16-byte aligned
    if (q_stride == 0) q_stride = (int64_t)H * D;
    if (out_stride == 0) out_stride = (int64_t)H * D;
    if (q_stride < (int64_t)H * D || out_stride < (int64_t)H * D) return PA_ERR_ARG;
    if ((q_stride | out_stride) & 7) return PA_ERR_ALIGN;
    WsLayout w = ws_layout(H, D, batch, 0, workspace_bytes);
    if (w.item_cap < batch || w.total > workspace_bytes) return PA_ERR_WORKSPACE;

    DeviceInfo dev;
    rc = get_device_info(&dev);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int* hdr = reinterpret_cast<int*>(ws);
    int* status = dev_status ? dev_status : hdr + HDR_STATUS;

    CUtensorMap km, vm;
    rc = make_cache_map(&km, k_cache, shape);
    if (rc) return rc;
    rc = make_cache_map(&vm, v_cache, shape);
    if (rc) return rc;

    DecodeParams dp;
    dp.q = static_cast<const __nv_bfloat16*>(q);
    dp.out = static_cast<__nv_bfloat16*>(out);
    dp.block_tables = block_tables;
    PlanAddr pa;
    pa.fixed = hdr;
    pa.region0 = ws + w.off_region;
    pa.region_bytes = w.region_bytes;
    pa.off_seqinfo = w.off_seqinfo;
    pa.off_multi = w.off_multi;
    pa.off_records = w.off_records;
    dp.plan = pa;
    dp.partial_o = reinterpret_cast<float*>(ws + w.off_o);
    dp.partial_ml = reinterpret_cast<float2*>(ws + w.off_ml);
    dp.status = status;
    dp.max_blocks = max_blocks_per_seq;
    dp.H = H;
    dp.Hkv = shape->num_kv_heads;
    dp.G = H / shape->num_kv_heads;
    dp.NB = shape->num_blocks;
    dp.scale_log2 = scale * 1.4426950408889634f;
    dp.q_stride = q_stride;
    dp.out_stride = out_stride;

    int total_warps = 0;
    rc = dispatch_decode(shape, km, vm, dp, dev, &total_warps, false, st, q_on_host);
    if (rc) return rc;

    ProfCall prof_ev;
    const bool prof = prof_begin_call(&prof_ev);
    if (prof) cudaEventRecord(prof_ev.ev[0], st);
    if (!(flags & PA_FLAG_REUSE_PLAN)) {
        PlanParams pp;
        pp.seq_lens = seq_lens;
        pp.batch = batch;
        pp.max_blocks = max_blocks_per_seq;
        pp.Hkv = shape->num_kv_heads;
        pp.H = H;
        pp.forced_p = partition_tokens;
        pp.no_direct = part != nullptr;
        pp.item_cap = w.item_cap;
        pp.total_warps = total_warps;
        pp.plan = pa;
        pp.status = status;
        count_launch();
        rc = check_cuda(launch_pdl(pa_plan_kernel, dim3(1), dim3(PLAN_THREADS), 0, st, pp));
        if (rc) return rc;
    }

    if (prof) cudaEventRecord(prof_ev.ev[1], st);
    rc = dispatch_decode(shape, km, vm, dp, dev, &total_warps, true, st, q_on_host);
    if (rc) return rc;
    if (prof) cudaEventRecord(prof_ev.ev[2], st);

    CombineParams cp = {};
    cp.plan = pa;
    cp.partial_o = dp.partial_o;
    cp.partial_ml = dp.partial_ml;
    cp.out = dp.out;
    cp.rows = batch * H;
    cp.H = H;
    cp.out_stride = out_stride;
    cp.counter_reset = 3 * total_warps;
    if (part) {
        cp.part_o = part;
        cp.part_ml = reinterpret_cast<float2*>(part + (size_t)cp.rows * D);
    }
    const int cgrid = cp.rows;
    count_launch();
    // One CTA fewer than the chip holds at once: the whole grid is resident together, so the
    // next call's plan kernel is launched as soon as this grid has started, and one SM keeps
    // threads and registers free for it.
    int per_sm = 0;
    rc = combine_rows_per_sm(D, &per_sm);
    if (rc) return rc;
    const dim3 rgrid(std::max(1, per_sm * dev.sm_count - 1)), rblock(256);
    rc = check_cuda(part       ? launch_combine<COMBINE_TO_PARTIAL>(D, cgrid, st, cp)
                    : D == 256 ? launch_pdl(pa_combine_rows_kernel<256>, rgrid, rblock, 0, st, cp)
                    : D == 128 ? launch_pdl(pa_combine_rows_kernel<128>, rgrid, rblock, 0, st, cp)
                               : launch_pdl(pa_combine_rows_kernel<64>, rgrid, rblock, 0, st, cp));
    if (prof) cudaEventRecord(prof_ev.ev[3], st);
    return rc;
}

extern "C" int pa_decode(const pa_shape* shape, const void* q, const void* k_cache,
                         const void* v_cache, const int32_t* block_tables,
                         int32_t max_blocks_per_seq, const int32_t* seq_lens, int32_t batch,
                         float scale, void* out, void* workspace, size_t workspace_bytes,
                         int32_t partition_tokens, int32_t flags, int32_t* dev_status,
                         void* cuda_stream) {
    return decode_impl(shape, q, k_cache, v_cache, block_tables, max_blocks_per_seq, seq_lens,
                       batch, scale, out, nullptr, workspace, workspace_bytes, partition_tokens,
                       flags, dev_status, cuda_stream);
}

extern "C" int pa_decode_strided(const pa_shape* shape, const void* q, int64_t q_stride_seq,
                                 const void* k_cache, const void* v_cache,
                                 const int32_t* block_tables, int32_t max_blocks_per_seq,
                                 const int32_t* seq_lens, int32_t batch, float scale, void* out,
                                 int64_t out_stride_seq, void* workspace, size_t workspace_bytes,
                                 int32_t partition_tokens, int32_t flags, int32_t* dev_status,
                                 void* cuda_stream) {
    if (q_stride_seq <= 0 || out_stride_seq <= 0) return PA_ERR_ARG;
    return decode_impl(shape, q, k_cache, v_cache, block_tables, max_blocks_per_seq, seq_lens,
                       batch, scale, out, nullptr, workspace, workspace_bytes, partition_tokens,
                       flags, dev_status, cuda_stream, q_stride_seq, out_stride_seq);
}

extern "C" int pa_partial_floats(const pa_shape* shape, int32_t batch, size_t* floats) {
    if (!shape || !floats) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (batch < 0) return PA_ERR_ARG;
    const size_t n = (size_t)batch * shape->num_q_heads * (shape->head_dim + 2);
    *floats = (n + 3) & ~(size_t)3;  // records packed back to back stay 16-byte aligned
    return PA_OK;
}

extern "C" int pa_decode_partial(const pa_shape* shape, const void* q, const void* k_cache,
                                 const void* v_cache, const int32_t* block_tables,
                                 int32_t max_blocks_per_seq, const int32_t* seq_lens,
                                 int32_t batch, float scale, float* part, void* workspace,
                                 size_t workspace_bytes, int32_t partition_tokens,
                                 int32_t* dev_status, void* cuda_stream) {
    if (batch > 0 && !part) return PA_ERR_NULL;
    return decode_impl(shape, q, k_cache, v_cache, block_tables, max_blocks_per_seq, seq_lens,
                       batch, scale, nullptr, part, workspace, workspace_bytes, partition_tokens,
                       0, dev_status, cuda_stream);
}

extern "C" int pa_merge_partials(const float* const* parts, int32_t num_parts, int32_t rows,
                                 int32_t head_dim, void* out, void* cuda_stream) {
    if (num_parts < 0 || num_parts > PA_MAX_PARTS || rows < 0) return PA_ERR_ARG;
    if (head_dim != 64 && head_dim != 128 && head_dim != 256) return PA_ERR_SHAPE;
    if (rows == 0) return PA_OK;
    if (!out || (num_parts > 0 && !parts)) return PA_ERR_NULL;
    if (!aligned16(out)) return PA_ERR_ALIGN;
    CombineParams cp = {};
    for (int i = 0; i < num_parts; ++i) {
        if (!parts[i]) return PA_ERR_NULL;
        if (!aligned16(parts[i])) return PA_ERR_ALIGN;
        cp.parts[i] = parts[i];
    }
    cp.out = static_cast<__nv_bfloat16*>(out);
    cp.rows = rows;
    cp.H = 1;
    cp.out_stride = head_dim;
    cp.n_parts = num_parts;
    DeviceInfo dev;
    int rc = get_device_info(&dev);
    if (rc) return rc;
    count_launch();
    return check_cuda(launch_combine<COMBINE_MERGE>(head_dim, rows, static_cast<cudaStream_t>(cuda_stream), cp));
}

extern "C" int pa_profile_enable(int on) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof_on = on != 0;
    return PA_OK;
}

extern "C" int pa_profile_read(double* plan_ms, double* attention_ms, double* combine_ms,
                               int64_t* calls) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    double t[3] = {0, 0, 0};
    int64_t n = 0;
    int rc = PA_OK;
    for (ProfCall& c : g_prof_calls) {
        if (rc == PA_OK) rc = check_cuda(cudaEventSynchronize(c.ev[3]));
        for (int i = 0; i < 3 && rc == PA_OK; ++i) {
            float ms = 0.f;
            rc = check_cuda(cudaEventElapsedTime(&ms, c.ev[i], c.ev[i + 1]));
            t[i] += ms;
        }
        if (rc == PA_OK) ++n;
        g_prof_free.push_back(c);
    }
    g_prof_calls.clear();
    if (plan_ms) *plan_ms = t[0];
    if (attention_ms) *attention_ms = t[1];
    if (combine_ms) *combine_ms = t[2];
    if (calls) *calls = n;
    return rc;
}

extern "C" int pa_host_io_bytes(const pa_shape* shape, int32_t max_batch,
                                int32_t max_blocks_per_seq, size_t* bytes) {
    if (!shape || !bytes) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (max_batch < 0 || max_blocks_per_seq < 0) return PA_ERR_ARG;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t qo = up((size_t)max_batch * shape->num_q_heads * shape->head_dim * 2);
    *bytes = 2 * qo + up((size_t)max_batch * max_blocks_per_seq * 4) + up((size_t)max_batch * 4);
    return PA_OK;
}

extern "C" int pa_decode_host(const pa_shape* shape, const void* q_host, const void* k_cache,
                              const void* v_cache, const int32_t* block_tables_host,
                              int32_t max_blocks_per_seq, const int32_t* seq_lens_host,
                              int32_t batch, float scale, void* out_host, void* io_buf,
                              size_t io_bytes, void* workspace, size_t workspace_bytes,
                              int32_t partition_tokens, int32_t* dev_status, void* cuda_stream) {
    if (!shape) return PA_ERR_NULL;
    int rc = validate_shape(shape);
    if (rc) return rc;
    if (batch < 0 || max_blocks_per_seq < 0) return PA_ERR_ARG;
    if (batch == 0) return PA_OK;
    if (!q_host || !block_tables_host || !seq_lens_host || !out_host || !io_buf)
        return PA_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(io_buf) & 255) return PA_ERR_ALIGN;
    size_t need = 0;
    rc = pa_host_io_bytes(shape, batch, max_blocks_per_seq, &need);
    if (rc) return rc;
    if (io_bytes < need) return PA_ERR_WORKSPACE;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t qbytes = (size_t)batch * shape->num_q_heads * shape->head_dim * 2;
    const size_t tbytes = (size_t)batch * max_blocks_per_seq * 4;
    uint8_t* io = static_cast<uint8_t*>(io_buf);
    void* dq = io;
    void* dout = io + up(qbytes);
    void* dtab = io + 2 * up(qbytes);
    void* dlen = io + 2 * up(qbytes) + up(tbytes);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // Pinned memory the GPU can address is used in place: block-table entries and the query
    // rows of a head group are fetched one to two work units ahead of their use (16 bytes per
    // lane, so that they cross the link as whole 128-byte reads), and output rows are posted as
    // they are produced: the transfers overlap the kernels instead of preceding / following
    // them.  q is re-read by every (partition, KV head) unit, a few times its size over the
    // link, which hides under the KV stream; groups of more than 8 heads and head_dim 256 copy
    // it once instead.
    auto mapped = [](const void* host) -> void* {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        return attr.type == cudaMemoryTypeHost ? attr.devicePointer : nullptr;
    };
    // a small table is cheaper to copy than to read entry by entry over the link
    void* tab_dev = tbytes >= (256u << 10) ? mapped(block_tables_host) : nullptr;
    void* out_dev = mapped(out_host);
    if (out_dev && (reinterpret_cast<uintptr_t>(out_dev) & 15)) out_dev = nullptr;
    void* q_dev = host_q_supported(shape) ? mapped(q_host) : nullptr;
    if (q_dev && (reinterpret_cast<uintptr_t>(q_dev) & 15)) q_dev = nullptr;
    if (q_dev) {
        // Every (partition, KV head) unit fetches its group's rows: worth it only while those
        // reads, at about 50 GB/s, fit well inside the time the KV stream takes at about
        // 6.4 TB/s; a batch of long sequences with many query heads re-reads q tens of times
        // and is better off with one copy.  The lengths are host data of this call.
        const int64_t P = partition_tokens ? partition_tokens : MAX_PART;
        const int64_t max_tok = (int64_t)max_blocks_per_seq * BS;
        int64_t tokens = 0, items = 0;
        for (int32_t b = 0; b < batch; ++b) {
            const int64_t L = seq_lens_host[b];
            if (L <= 0 || L > max_tok) continue;
            tokens += L;
            items += (L + P - 1) / P;
        }
        const int G = shape->num_q_heads / shape->num_kv_heads;
        const double q_us = (double)items * shape->num_kv_heads * G * shape->head_dim * 2 / 50e3;
        const double kv_us = (double)tokens * 2 * shape->num_kv_heads * shape->head_dim * 2 / 6.4e6;
        if (q_us > 0.65 * kv_us) q_dev = nullptr;
    }
    const bool q_in_place = q_dev != nullptr;
    if (!q_in_place) {
        rc = check_cuda(cudaMemcpyAsync(dq, q_host, qbytes, cudaMemcpyHostToDevice, st));
        if (rc) return rc;
        q_dev = dq;
    }
    if (!tab_dev) {
        rc = check_cuda(
            cudaMemcpyAsync(dtab, block_tables_host, tbytes, cudaMemcpyHostToDevice, st));
        if (rc) return rc;
        tab_dev = dtab;
    }
    rc = check_cuda(
        cudaMemcpyAsync(dlen, seq_lens_host, (size_t)batch * 4, cudaMemcpyHostToDevice, st));
    if (rc) return rc;
    rc = decode_impl(shape, q_dev, k_cache, v_cache, static_cast<const int32_t*>(tab_dev),
                     max_blocks_per_seq, static_cast<const int32_t*>(dlen), batch, scale,
                     out_dev ? out_dev : dout, nullptr, workspace, workspace_bytes,
                     partition_tokens, 0, dev_status, cuda_stream, 0, 0, q_in_place);
    if (rc || out_dev) return rc;
    return check_cuda(cudaMemcpyAsync(out_host, dout, qbytes, cudaMemcpyDeviceToHost, st));
}

// ======================================================================================
// pa_decode_static: the same three kernels, scratch taken from a fixed device array
// ======================================================================================
// The array below is part of the loaded module: every GPU that loads this library sets
// PA_STATIC_WORKSPACE_BYTES aside for it until the process exits.  In host code the name
// `g_static_workspace` is only a handle for the runtime; the device address that kernels
// can use comes from cudaGetSymbolAddress, asked once per device with that device current.
static __device__ __align__(256) unsigned char g_static_workspace[PA_STATIC_WORKSPACE_BYTES];

static int static_workspace_address(void** out) {
    static std::mutex mu;
    static void* addr[64] = {nullptr};
    int dev = 0;
    int rc = pk::check_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    if (dev < 0 || dev >= 64) return PA_ERR_ARG;
    std::lock_guard<std::mutex> lk(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        rc = pk::check_cuda(cudaGetSymbolAddress(&p, g_static_workspace));
        if (rc) return rc;
        if (!p) return PA_ERR_CUDA;
        addr[dev] = p;
    }
    *out = addr[dev];
    return PA_OK;
}

extern "C" int pa_decode_static(const pa_shape* shape, const void* q, const void* k_cache,
                                const void* v_cache, const int32_t* block_tables,
                                int32_t max_blocks_per_seq, const int32_t* seq_lens,
                                int32_t batch, int64_t max_total_tokens, float scale, void* out,
                                int32_t partition_tokens, int32_t* dev_status,
                                void* cuda_stream) {
    size_t need = 0;
    int rc = pa_workspace_bytes(shape, batch, max_total_tokens, partition_tokens, &need);
    if (rc) return rc;
    if (need > (size_t)PA_STATIC_WORKSPACE_BYTES) return PA_ERR_STATIC_LIMIT;
    if (batch == 0) return PA_OK;
    void* ws = nullptr;
    rc = static_workspace_address(&ws);
    if (rc) return rc;
    // the array still holds the previous call's plan header and fallback status word
    rc = pk::check_cuda(cudaMemsetAsync(ws, 0, pk::HDR_WORDS * sizeof(int),
                                        static_cast<cudaStream_t>(cuda_stream)));
    if (rc) return rc;
    return pa_decode(shape, q, k_cache, v_cache, block_tables, max_blocks_per_seq, seq_lens, batch,
                     scale, out, ws, (size_t)PA_STATIC_WORKSPACE_BYTES, partition_tokens, 0,
                     dev_status, cuda_stream);
}
