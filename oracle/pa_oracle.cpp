// CPU oracle for paged-attention decode and KV-block swaps.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain definition that the CUDA library is checked against.  It
// shares no code, header, table or helper with the CUDA path and must never be called by
// it; only the tests, the smoke check and the benchmark's CPU-baseline leg load it.
//
// What it computes.
//   Decode (Section 2.1 "Decoding": each step uses the KV-Cache of all previous tokens;
//   Section 2.2 "KV-Cache": the cache is cut into fixed-size blocks that are not
//   contiguous in physical memory and are reached through a logical-to-physical map;
//   Section 4.2, Eq. 3: the kernel streams the whole KV history of every running
//   sequence at every step).  For sequence b with L = seq_lens[b] cached tokens and
//   query head h (KV head h / G, G = H / Hkv):
//        s_t  = scale * sum_d q[b,h,d] * K[p(t), kvh, t mod bs, d],  p(t) = table[b][t / bs]
//        m    = max_t s_t,  w_t = exp(s_t - m),  Z = sum_t w_t
//        out[b,h,d] = sum_t w_t * V[p(t), kvh, t mod bs, d] / Z
//   All operands are widened exactly from bf16 to double; nothing is blocked, split or
//   reordered.  Slots at or beyond L and table entries beyond ceil(L / bs) are never
//   read.  L = 0 gives a row of zeros (the paper does not define it; this is the
//   library's stated contract).
//   Swap (Section 5.1.2 "Swapping": the victim's KV blocks move to host memory and later
//   come back into newly allocated blocks): a byte copy of whole blocks, all layers,
//   K then V, into / out of a contiguous host image laid out
//   [block i][layer][K|V][kv head][slot][dim].
//   Append (Section 2.2): the new token's K/V rows are written into their slot.
//   Prefill (Sections 2.1, 5.1.2 "Recomputation"): causal attention of a chunk of query
//   tokens over the paged cache, the definition above applied per query position.
//
// Pins (tests, CPU only): brute-force dense attention without max subtraction in long
// double on un-paged copies, closed forms (L = 1, L = 2 logistic weights, equal keys ->
// mean of V, a dominant key, score-shift invariance), invariants (physical permutation,
// batch composition, GQA == MHA with replicated KV heads), poison in unused slots, and
// planted-mistake checks.  Nothing here is "parity unpinned".
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline double bf16_to_double(uint16_t bits) {
    uint32_t u = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

}  // namespace

extern "C" {

// Number of worker threads the decode oracle will use for `requested` (0 = all).
int oracle_threads(int requested) {
#ifdef _OPENMP
    int n = omp_get_max_threads();
    if (requested > 0 && requested < n) n = requested;
    return n;
#else
    (void)requested;
    return 1;
#endif
}

// out: double [batch, H, D].  Strides are in elements of the bf16 pools; the last
// dimension (dim) has stride 1.  Returns 0, or -1 on an invalid length / block id (the
// oracle refuses rather than reading outside the pool).
int oracle_pa_decode(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                     const int32_t* block_tables, int32_t max_blocks, const int32_t* seq_lens,
                     int32_t batch, int32_t H, int32_t Hkv, int32_t D, int32_t bs,
                     int32_t num_blocks, int64_t stride_block, int64_t stride_head,
                     int64_t stride_tok, double scale, double* out, int32_t num_threads) {
    if (H % Hkv != 0) return -1;
    const int G = H / Hkv;
    for (int b = 0; b < batch; ++b) {
        const int L = seq_lens[b];
        if (L < 0 || L > static_cast<int64_t>(max_blocks) * bs) return -1;
        for (int j = 0; j < (L + bs - 1) / bs; ++j) {
            const int p = block_tables[static_cast<int64_t>(b) * max_blocks + j];
            if (p < 0 || p >= num_blocks) return -1;
        }
    }
    const int64_t rows = static_cast<int64_t>(batch) * H;
#ifdef _OPENMP
    const int nt = oracle_threads(num_threads);
#pragma omp parallel for schedule(dynamic, 1) num_threads(nt)
#else
    (void)num_threads;
#endif
    for (int64_t r = 0; r < rows; ++r) {
        const int b = static_cast<int>(r / H);
        const int h = static_cast<int>(r % H);
        const int kvh = h / G;
        const int L = seq_lens[b];
        double* o = out + r * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (L == 0) continue;
        const uint16_t* qrow = q + r * D;
        const int32_t* table = block_tables + static_cast<int64_t>(b) * max_blocks;
        std::vector<double> s(L);
        // scores
        for (int t = 0; t < L; ++t) {
            const int64_t base = table[t / bs] * stride_block + kvh * stride_head +
                                 (t % bs) * stride_tok;
            double acc = 0.0;
            for (int d = 0; d < D; ++d)
                acc += bf16_to_double(qrow[d]) * bf16_to_double(k_cache[base + d]);
            s[t] = scale * acc;
        }
        // softmax weights
        double m = s[0];
        for (int t = 1; t < L; ++t) m = s[t] > m ? s[t] : m;
        double Z = 0.0;
        for (int t = 0; t < L; ++t) {
            s[t] = std::exp(s[t] - m);
            Z += s[t];
        }
        // weighted sum of values
        for (int t = 0; t < L; ++t) {
            const int64_t base = table[t / bs] * stride_block + kvh * stride_head +
                                 (t % bs) * stride_tok;
            const double w = s[t];
            for (int d = 0; d < D; ++d) o[d] += w * bf16_to_double(v_cache[base + d]);
        }
        for (int d = 0; d < D; ++d) o[d] /= Z;
    }
    return 0;
}

// Host image of n evicted blocks: [i][layer][K|V][kv head][slot][dim], bf16 bit patterns.
// k_pool / v_pool hold all layers; layer l of K starts at k_pool + l * layer_stride_k.
int oracle_swap_out(const uint16_t* k_pool, const uint16_t* v_pool, int32_t num_layers,
                    int64_t layer_stride_k, int64_t layer_stride_v, int32_t Hkv, int32_t D,
                    int32_t bs, int32_t num_blocks, int64_t stride_block, int64_t stride_head,
                    int64_t stride_tok, const int32_t* block_ids, int32_t n, uint16_t* host) {
    int64_t o = 0;
    for (int i = 0; i < n; ++i) {
        const int p = block_ids[i];
        if (p < 0 || p >= num_blocks) return -1;
        for (int l = 0; l < num_layers; ++l)
            for (int kv = 0; kv < 2; ++kv) {
                const uint16_t* pool = kv == 0 ? k_pool + l * layer_stride_k
                                               : v_pool + l * layer_stride_v;
                for (int h = 0; h < Hkv; ++h)
                    for (int t = 0; t < bs; ++t)
                        for (int d = 0; d < D; ++d)
                            host[o++] = pool[p * stride_block + h * stride_head +
                                             t * stride_tok + d];
            }
    }
    return 0;
}

// Inverse of oracle_swap_out: host slot i is written into physical block block_ids[i].
// Every pool element outside the listed blocks is left untouched.
int oracle_swap_in(uint16_t* k_pool, uint16_t* v_pool, int32_t num_layers,
                   int64_t layer_stride_k, int64_t layer_stride_v, int32_t Hkv, int32_t D,
                   int32_t bs, int32_t num_blocks, int64_t stride_block, int64_t stride_head,
                   int64_t stride_tok, const int32_t* block_ids, int32_t n,
                   const uint16_t* host) {
    int64_t o = 0;
    for (int i = 0; i < n; ++i) {
        const int p = block_ids[i];
        if (p < 0 || p >= num_blocks) return -1;
        for (int l = 0; l < num_layers; ++l)
            for (int kv = 0; kv < 2; ++kv) {
                uint16_t* pool = kv == 0 ? k_pool + l * layer_stride_k
                                         : v_pool + l * layer_stride_v;
                for (int h = 0; h < Hkv; ++h)
                    for (int t = 0; t < bs; ++t)
                        for (int d = 0; d < D; ++d)
                            pool[p * stride_block + h * stride_head + t * stride_tok + d] =
                                host[o++];
            }
    }
    return 0;
}

// KV append (Section 2.2 "KV-Cache": with every decoding step the new token's K and V
// vectors are appended to the cache).  Token b goes to flat slot slot_mapping[b] =
// block * bs + offset of one layer's cache; a negative slot means "no token" (padding).
// Returns -1 (nothing guaranteed written) if a slot is beyond the pool.
int oracle_kv_append(uint16_t* k_cache, uint16_t* v_cache, const uint16_t* k_new,
                     const uint16_t* v_new, const int64_t* slot_mapping, int32_t batch,
                     int32_t Hkv, int32_t D, int32_t bs, int32_t num_blocks, int64_t stride_block,
                     int64_t stride_head, int64_t stride_tok) {
    for (int b = 0; b < batch; ++b)
        if (slot_mapping[b] >= static_cast<int64_t>(num_blocks) * bs) return -1;
    for (int b = 0; b < batch; ++b) {
        const int64_t slot = slot_mapping[b];
        if (slot < 0) continue;
        const int64_t p = slot / bs, t = slot % bs;
        for (int h = 0; h < Hkv; ++h)
            for (int d = 0; d < D; ++d) {
                const int64_t dst = p * stride_block + h * stride_head + t * stride_tok + d;
                const int64_t src = (static_cast<int64_t>(b) * Hkv + h) * D + d;
                k_cache[dst] = k_new[src];
                v_cache[dst] = v_new[src];
            }
    }
    return 0;
}

// Prefill / recomputation attention (Section 2.1 "Prefill": the prompt is processed in
// parallel; Section 5.1.2 "Recomputation": a preempted request's prompt and generated tokens
// are re-processed from scratch; Appendix B.1: prefill is scheduled in chunks).  Sequence b
// contributes q_len_b = cu_q_lens[b+1] - cu_q_lens[b] query tokens, the last q_len_b of its
// ctx_lens[b] cached tokens (their K/V are already in the cache).  Query i sits at position
// pos = ctx_b - q_len_b + i and attends causally to cached tokens t <= pos:
//     out[cu_q_lens[b] + i, h, :] = softmax_{t <= pos}(scale * <q, K_t>) . V_t
// out: double [total_q, H, D].  Returns -1 on inconsistent lengths or a bad block id.
int oracle_pa_prefill(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                      const int32_t* block_tables, int32_t max_blocks, const int32_t* ctx_lens,
                      const int32_t* cu_q_lens, int32_t batch, int32_t H, int32_t Hkv, int32_t D,
                      int32_t bs, int32_t num_blocks, int64_t stride_block, int64_t stride_head,
                      int64_t stride_tok, double scale, double* out, int32_t num_threads) {
    if (H % Hkv != 0) return -1;
    const int G = H / Hkv;
    if (batch > 0 && cu_q_lens[0] != 0) return -1;
    for (int b = 0; b < batch; ++b) {
        const int ql = cu_q_lens[b + 1] - cu_q_lens[b], L = ctx_lens[b];
        if (ql < 0 || L < ql || L > static_cast<int64_t>(max_blocks) * bs) return -1;
        for (int j = 0; j < (L + bs - 1) / bs; ++j) {
            const int p = block_tables[static_cast<int64_t>(b) * max_blocks + j];
            if (p < 0 || p >= num_blocks) return -1;
        }
    }
    const int total_q = batch > 0 ? cu_q_lens[batch] : 0;
    std::vector<int> seq_of(total_q);
    for (int b = 0; b < batch; ++b)
        for (int i = cu_q_lens[b]; i < cu_q_lens[b + 1]; ++i) seq_of[i] = b;
    const int64_t rows = static_cast<int64_t>(total_q) * H;
#ifdef _OPENMP
    const int nt = oracle_threads(num_threads);
#pragma omp parallel for schedule(dynamic, 1) num_threads(nt)
#else
    (void)num_threads;
#endif
    for (int64_t r = 0; r < rows; ++r) {
        const int tok = static_cast<int>(r / H), h = static_cast<int>(r % H), kvh = h / G;
        const int b = seq_of[tok];
        const int ql = cu_q_lens[b + 1] - cu_q_lens[b];
        const int pos = ctx_lens[b] - ql + (tok - cu_q_lens[b]);
        const int n = pos + 1;  // visible cached tokens
        double* o = out + r * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        const uint16_t* qrow = q + r * D;
        const int32_t* table = block_tables + static_cast<int64_t>(b) * max_blocks;
        std::vector<double> s(n);
        for (int t = 0; t < n; ++t) {
            const int64_t base = table[t / bs] * stride_block + kvh * stride_head +
                                 (t % bs) * stride_tok;
            double acc = 0.0;
            for (int d = 0; d < D; ++d)
                acc += bf16_to_double(qrow[d]) * bf16_to_double(k_cache[base + d]);
            s[t] = scale * acc;
        }
        double m = s[0];
        for (int t = 1; t < n; ++t) m = s[t] > m ? s[t] : m;
        double Z = 0.0;
        for (int t = 0; t < n; ++t) {
            s[t] = std::exp(s[t] - m);
            Z += s[t];
        }
        for (int t = 0; t < n; ++t) {
            const int64_t base = table[t / bs] * stride_block + kvh * stride_head +
                                 (t % bs) * stride_tok;
            const double w = s[t];
            for (int d = 0; d < D; ++d) o[d] += w * bf16_to_double(v_cache[base + d]);
        }
        for (int d = 0; d < D; ++d) o[d] /= Z;
    }
    return 0;
}

}  // extern "C"
