// One 16-token KV block against a 16-row query fragment: S = Q K^T, online softmax, O += P V.
// Shared by the decode and the prefill kernels.  The K and V tiles sit in shared memory as
// TMA wrote them: per 64-dim half, 16 rows of 128 bytes with the 128-byte swizzle.
#pragma once
#include "ptx.cuh"

namespace pk {

// SPLITW: each softmax weight goes to the MMA as two bf16 numbers, its rounded value and the
// rounded remainder, so the weights carry about 16 significant bits and the result differs
// from the exact weighted mean by the output's own rounding only.  It doubles the P V MMAs.
template <int D, bool HI, bool SPLITW = false>
struct AttnFrag {
    static constexpr int KS = D / 16;      // k-steps of Q K^T
    static constexpr int NT = D / 8;       // n-tiles of O
    static constexpr int QW = HI ? 4 : 2;  // A-fragment words per k-step (rows g and g+8)
    static constexpr int HALF_BYTES = 16 * 128;

    // running state of rows g (index 0) and g + 8 (index 1); o is un-normalised
    float o[NT][4];
    float m0, m1, l0, l1;
    // per-lane pieces of the ldmatrix addresses
    uint32_t k_row, k_cb, v_row, v_cb, mr;
    int t;

    __device__ __forceinline__ void init_lane(int lane) {
        // K (B operand, not transposed): matrix i = lane>>3 -> tokens (i>>1)*8.., 16-byte chunk
        // 2*ks + (i&1); V (B operand, transposed): tokens (i&1)*8.., chunk 2*jj + (i>>1).
        const int mi = lane >> 3;
        mr = lane & 7;
        k_row = ((mi >> 1) * 8 + mr) * 128;
        k_cb = mi & 1;
        v_row = ((mi & 1) * 8 + mr) * 128;
        v_cb = mi >> 1;
        t = lane & 3;
    }
    __device__ __forceinline__ void reset() {
        m0 = m1 = -INFINITY;
        l0 = l1 = 0.f;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    }

    // kbase / vbase: shared addresses of the K and V tiles.  qa: A fragments of Q.
    // lim0 / lim1: number of leading tokens of this block that rows g / g+8 may see (0..16).
    // nstore: tokens of this block that hold data at all (slots past the end of the sequence
    // may contain anything and get their V rows zeroed).  sl2 = scale * log2(e).
    __device__ __forceinline__ void attend(uint32_t kbase, uint32_t vbase,
                                           const uint32_t (&qa)[KS][QW], int lim0, int lim1,
                                           int nstore, float sl2, int lane) {
        if (nstore < 16) {
            // 0 * NaN would poison the accumulators; scores of those slots are masked below
            const int nchunk = (16 - nstore) * 8;
            for (int hf = 0; hf < D / 64; ++hf)
                for (int c = lane; c < nchunk; c += 32)
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(
                                     vbase + hf * HALF_BYTES + nstore * 128 + c * 16),
                                 "r"(0u)
                                 : "memory");
            fence_proxy_async_smem();
            __syncwarp();
        }

        // S = Q K^T for 16 tokens: two n-tiles of 8 tokens
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t b00, b01, b10, b11;
            const uint32_t chunk = ((ks & 3) * 2 + k_cb) ^ mr;
            ldmatrix_x4(kbase + (ks >> 2) * HALF_BYTES + k_row + (chunk << 4), b00, b01, b10, b11);
            const uint32_t a0 = qa[ks][0], a2 = qa[ks][QW == 4 ? 2 : 1];
            const uint32_t a1 = HI ? qa[ks][1] : 0u, a3 = HI ? qa[ks][QW - 1] : 0u;
            mma_bf16_16816(s0, a0, a1, a2, a3, b00, b01);
            mma_bf16_16816(s1, a0, a1, a2, a3, b10, b11);
        }

        // scale to log2 units, mask tokens the row may not see
        const int c0 = 2 * t;
        s0[0] = c0 < lim0 ? s0[0] * sl2 : -INFINITY;
        s0[1] = c0 + 1 < lim0 ? s0[1] * sl2 : -INFINITY;
        s1[0] = c0 + 8 < lim0 ? s1[0] * sl2 : -INFINITY;
        s1[1] = c0 + 9 < lim0 ? s1[1] * sl2 : -INFINITY;
        float mx0 = fmaxf(fmaxf(s0[0], s0[1]), fmaxf(s1[0], s1[1]));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        const float mn0 = fmaxf(m0, mx0);
        const float mu0 = mn0 == -INFINITY ? 0.f : mn0;
        const float corr0 = ex2(m0 - mu0);
        m0 = mn0;
        const float e00 = ex2(s0[0] - mu0), e01 = ex2(s0[1] - mu0);
        const float e10 = ex2(s1[0] - mu0), e11 = ex2(s1[1] - mu0);
        const uint32_t pa0 = pack_bf16x2(e00, e01);
        const uint32_t pa2 = pack_bf16x2(e10, e11);
        uint32_t pb0 = 0u, pb1 = 0u, pb2 = 0u, pb3 = 0u;
        if (SPLITW) {
            pb0 = pack_bf16x2(e00 - bf16lo_to_f32(pa0), e01 - bf16hi_to_f32(pa0));
            pb2 = pack_bf16x2(e10 - bf16lo_to_f32(pa2), e11 - bf16hi_to_f32(pa2));
            l0 = l0 * corr0 + ((e00 + e01) + (e10 + e11));
        } else {
            // the row sum uses the rounded weights, the same ones the MMA multiplies by
            l0 = l0 * corr0 + ((bf16lo_to_f32(pa0) + bf16hi_to_f32(pa0)) +
                               (bf16lo_to_f32(pa2) + bf16hi_to_f32(pa2)));
        }
        uint32_t pa1 = 0u, pa3 = 0u;
        float corr1 = 1.f;
        if (HI) {
            s0[2] = c0 < lim1 ? s0[2] * sl2 : -INFINITY;
            s0[3] = c0 + 1 < lim1 ? s0[3] * sl2 : -INFINITY;
            s1[2] = c0 + 8 < lim1 ? s1[2] * sl2 : -INFINITY;
            s1[3] = c0 + 9 < lim1 ? s1[3] * sl2 : -INFINITY;
            float mx1 = fmaxf(fmaxf(s0[2], s0[3]), fmaxf(s1[2], s1[3]));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float mn1 = fmaxf(m1, mx1);
            const float mu1 = mn1 == -INFINITY ? 0.f : mn1;
            corr1 = ex2(m1 - mu1);
            m1 = mn1;
            const float f00 = ex2(s0[2] - mu1), f01 = ex2(s0[3] - mu1);
            const float f10 = ex2(s1[2] - mu1), f11 = ex2(s1[3] - mu1);
            pa1 = pack_bf16x2(f00, f01);
            pa3 = pack_bf16x2(f10, f11);
            if (SPLITW) {
                pb1 = pack_bf16x2(f00 - bf16lo_to_f32(pa1), f01 - bf16hi_to_f32(pa1));
                pb3 = pack_bf16x2(f10 - bf16lo_to_f32(pa3), f11 - bf16hi_to_f32(pa3));
                l1 = l1 * corr1 + ((f00 + f01) + (f10 + f11));
            } else {
                l1 = l1 * corr1 + ((bf16lo_to_f32(pa1) + bf16hi_to_f32(pa1)) +
                                   (bf16lo_to_f32(pa3) + bf16hi_to_f32(pa3)));
            }
        }
        // rescale only when some row's maximum moved (warp-uniform branch)
        if (__any_sync(0xffffffffu, corr0 != 1.f || corr1 != 1.f)) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                o[nt][0] *= corr0;
                o[nt][1] *= corr0;
                if (HI) {
                    o[nt][2] *= corr1;
                    o[nt][3] *= corr1;
                }
            }
        }

        // O += P V: V^T fragments straight from the [token][dim] tile
#pragma unroll
        for (int jj = 0; jj < D / 16; ++jj) {
            uint32_t v0, v1, v2, v3;
            const uint32_t chunk = ((jj & 3) * 2 + v_cb) ^ mr;
            ldmatrix_x4_trans(vbase + (jj >> 2) * HALF_BYTES + v_row + (chunk << 4), v0, v1, v2,
                              v3);
            mma_bf16_16816(o[2 * jj], pa0, pa1, pa2, pa3, v0, v1);
            mma_bf16_16816(o[2 * jj + 1], pa0, pa1, pa2, pa3, v2, v3);
            if (SPLITW) {
                mma_bf16_16816(o[2 * jj], pb0, pb1, pb2, pb3, v0, v1);
                mma_bf16_16816(o[2 * jj + 1], pb0, pb1, pb2, pb3, v2, v3);
            }
        }
    }

    // row sums are kept per thread; add the four threads of a row's quad
    __device__ __forceinline__ void reduce_row_sums() {
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        if (HI) {
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        }
    }
};

// The same block step for groups of at most 8 query heads, with the roles of the MMA operands
// exchanged: S^T = K Q^T has the 16 tokens of the block as its rows and the heads as its 8
// columns, O^T = V^T P^T the head dims as rows.  Nothing of the 16 x 8 tiles is padding, so a
// block takes half the MMAs of AttnFrag and the output accumulator half the registers (64 per
// thread at head_dim 256).  The Q fragments are the ones AttnFrag uses (its A fragment of rows
// 0..7 is this B fragment); the K and V tiles are read with the same ldmatrix addresses.
// A thread holds, of S^T, tokens g and g + 8 for heads 2t and 2t + 1 (g = lane / 4,
// t = lane % 4); the softmax statistics of a head are shared by the eight lanes with equal t.
template <int D, bool SPLITW = false>
struct AttnFragT {
    static constexpr int KS = D / 16;      // k-steps of K Q^T
    static constexpr int MT = D / 16;      // 16-dim row tiles of O^T
    static constexpr int HALF_BYTES = 16 * 128;

    // o[jj]: dims 16 jj + g (0, 1) and 16 jj + g + 8 (2, 3) for heads 2t (0, 2) and 2t + 1 (1, 3)
    float o[MT][4];
    float m0, m1, l0, l1;  // heads 2t and 2t + 1; l is this thread's share until reduce_row_sums
    uint32_t k_row, k_cb, v_row, v_cb, mr;
    int g;

    __device__ __forceinline__ void init_lane(int lane) {
        const int mi = lane >> 3;
        mr = lane & 7;
        k_row = ((mi >> 1) * 8 + mr) * 128;
        k_cb = mi & 1;
        v_row = ((mi & 1) * 8 + mr) * 128;
        v_cb = mi >> 1;
        g = lane >> 2;
    }
    __device__ __forceinline__ void reset() {
        m0 = m1 = -INFINITY;
        l0 = l1 = 0.f;
#pragma unroll
        for (int jj = 0; jj < MT; ++jj) o[jj][0] = o[jj][1] = o[jj][2] = o[jj][3] = 0.f;
    }

    // Arguments as for AttnFrag::attend; every head of a decode step sees the same tokens, so
    // one limit serves (lim1 is ignored).
    __device__ __forceinline__ void attend(uint32_t kbase, uint32_t vbase,
                                           const uint32_t (&qb)[KS][2], int lim, int /*lim1*/,
                                           int nstore, float sl2, int lane) {
        if (nstore < 16) {
            const int nchunk = (16 - nstore) * 8;
            for (int hf = 0; hf < D / 64; ++hf)
                for (int c = lane; c < nchunk; c += 32)
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(
                                     vbase + hf * HALF_BYTES + nstore * 128 + c * 16),
                                 "r"(0u)
                                 : "memory");
            fence_proxy_async_smem();
            __syncwarp();
        }

        // S^T = K Q^T: the four 8 x 8 pieces of the K tile are the A fragment
        float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t k00, k01, k10, k11;  // (tokens 0-7 | 8-15) x (dims 0-7 | 8-15) of the k-step
            const uint32_t chunk = ((ks & 3) * 2 + k_cb) ^ mr;
            ldmatrix_x4(kbase + (ks >> 2) * HALF_BYTES + k_row + (chunk << 4), k00, k01, k10, k11);
            mma_bf16_16816(s, k00, k10, k01, k11, qb[ks][0], qb[ks][1]);
        }

        // log2 units, tokens past the limit masked; the maximum of a head over the 16 tokens
        s[0] = g < lim ? s[0] * sl2 : -INFINITY;
        s[1] = g < lim ? s[1] * sl2 : -INFINITY;
        s[2] = g + 8 < lim ? s[2] * sl2 : -INFINITY;
        s[3] = g + 8 < lim ? s[3] * sl2 : -INFINITY;
        float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
        for (int d = 4; d <= 16; d <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, d));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, d));
        }
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
        const float corr0 = ex2(m0 - mu0), corr1 = ex2(m1 - mu1);
        m0 = mn0;
        m1 = mn1;
        const float e0 = ex2(s[0] - mu0), e1 = ex2(s[1] - mu1);
        const float e2 = ex2(s[2] - mu0), e3 = ex2(s[3] - mu1);
        // P as stored: (token g | g + 8) x (heads 2t, 2t + 1); as the B operand of O^T = V^T P^T
        // it is needed transposed, (tokens 2t, 2t + 1) x head g
        const uint32_t pa = pack_bf16x2(e0, e1), pc = pack_bf16x2(e2, e3);
        const uint32_t b0 = movmatrix_trans(pa), b1 = movmatrix_trans(pc);
        uint32_t r0 = 0u, r1 = 0u;
        if (SPLITW) {
            r0 = movmatrix_trans(pack_bf16x2(e0 - bf16lo_to_f32(pa), e1 - bf16hi_to_f32(pa)));
            r1 = movmatrix_trans(pack_bf16x2(e2 - bf16lo_to_f32(pc), e3 - bf16hi_to_f32(pc)));
            l0 = l0 * corr0 + (e0 + e2);
            l1 = l1 * corr1 + (e1 + e3);
        } else {
            l0 = l0 * corr0 + (bf16lo_to_f32(pa) + bf16lo_to_f32(pc));
            l1 = l1 * corr1 + (bf16hi_to_f32(pa) + bf16hi_to_f32(pc));
        }
        if (__any_sync(0xffffffffu, corr0 != 1.f || corr1 != 1.f)) {
#pragma unroll
            for (int jj = 0; jj < MT; ++jj) {
                o[jj][0] *= corr0;
                o[jj][1] *= corr1;
                o[jj][2] *= corr0;
                o[jj][3] *= corr1;
            }
        }

        // O^T += V^T P^T: the transposed 8 x 8 pieces of the V tile are the A fragment
#pragma unroll
        for (int jj = 0; jj < MT; ++jj) {
            uint32_t v0, v1, v2, v3;  // (dims 0-7: tokens 0-7, 8-15), (dims 8-15: tokens 0-7, 8-15)
            const uint32_t chunk = ((jj & 3) * 2 + v_cb) ^ mr;
            ldmatrix_x4_trans(vbase + (jj >> 2) * HALF_BYTES + v_row + (chunk << 4), v0, v1, v2,
                              v3);
            mma_bf16_16816(o[jj], v0, v2, v1, v3, b0, b1);
            if (SPLITW) mma_bf16_16816(o[jj], v0, v2, v1, v3, r0, r1);
        }
    }

    // the eight lanes with equal t hold the shares of a head's row sum
    __device__ __forceinline__ void reduce_row_sums() {
#pragma unroll
        for (int d = 4; d <= 16; d <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, d);
            l1 += __shfl_xor_sync(0xffffffffu, l1, d);
        }
    }
};

}  // namespace pk
