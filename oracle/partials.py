"""fp64 oracle of the sequence-split decode: per-slice partial results and their merge.
TEST INFRASTRUCTURE ONLY (numpy, plain loops over sequences; imports nothing from the CUDA
package).

The definition followed: attention of one query over a set of tokens T is
sum_{t in T} e^{s_t} V_t / sum_{t in T} e^{s_t}.  For a disjoint union T = T_1 u ... u T_R,
numerator and denominator are sums over the parts; each part is kept relative to its own
maximum m_i (natural-log units here), so the union is
sum_i e^{m_i - M} o_i / sum_i e^{m_i - M} l_i with M = max_i m_i.
The decode path it shards streams the whole KV history of a sequence every step (Section 4.2,
Eq. 3); tensor-parallel deployments of Section 6.4 are the setting in which a context is
spread over several GPUs.
"""
from __future__ import annotations

import numpy as np


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def decode_partial(q, k_cache, v_cache, block_tables, seq_lens, scale):
    """(o[B,H,D], m[B,H], l[B,H]) of every query row over the first seq_lens[b] tokens reached
    through block_tables[b]: m = max_t s_t (-inf for an empty slice), l = sum_t e^(s_t - m),
    o = sum_t e^(s_t - m) V_t, s_t = scale * <q, K_t>.  Inputs are bf16 bit patterns."""
    B, H, D = q.shape
    NB, Hkv, bs, _ = k_cache.shape
    G = H // Hkv
    qf = _bf16_to_f64(q)
    sigma = float(np.float32(scale))
    o = np.zeros((B, H, D))
    m = np.full((B, H), -np.inf)
    l = np.zeros((B, H))
    for b in range(B):
        L = int(seq_lens[b])
        if L == 0:
            continue
        t = np.arange(L)
        blk = np.asarray(block_tables[b])[t // bs].astype(np.int64)
        if (blk < 0).any() or (blk >= NB).any():
            raise ValueError("block id outside the pool")
        slot = t % bs
        for kvh in range(Hkv):
            K = _bf16_to_f64(k_cache[blk, kvh, slot, :])  # [L, D]
            V = _bf16_to_f64(v_cache[blk, kvh, slot, :])
            for h in range(kvh * G, (kvh + 1) * G):
                s = sigma * (K @ qf[b, h])
                mx = s.max()
                w = np.exp(s - mx)
                m[b, h] = mx
                l[b, h] = w.sum()
                o[b, h] = w @ V
    return o, m, l


def merge_partials(parts):
    """out[B,H,D] from a list of (o, m, l) triples; a row that is empty in every part is zeros."""
    ms = np.stack([p[1] for p in parts])  # [R, B, H]
    M = ms.max(axis=0)
    M = np.where(np.isinf(M), 0.0, M)
    num = np.zeros_like(parts[0][0])
    den = np.zeros_like(parts[0][2])
    for o, m, l in parts:
        w = np.exp(m - M)  # e^(-inf) = 0 for an empty part
        num += w[..., None] * o
        den += w * l
    out = np.zeros_like(num)
    nz = den > 0
    out[nz] = num[nz] / den[nz][..., None]
    return out
