"""Pins of the prefill oracle: brute-force dense causal attention (long double, masked
matrix form), equality with the already pinned decode oracle position by position, chunking
invariance, and planted mistakes."""
import numpy as np
import pytest

import oracle
from paper_2602_07878_b200 import workloads as wl


def make_case(ctx, qlens, H=4, Hkv=2, D=64, seed=1):
    spec = wl.make_spec("t", seq_lens=ctx, num_q_heads=H, num_kv_heads=Hkv, head_dim=D,
                        occupancy=0.8, seed=seed)
    k, v = wl.pools_np(spec)
    cu = np.concatenate([[0], np.cumsum(qlens)]).astype(np.int32)
    q = wl.normal_bf16_np(0, int(cu[-1]) * H * D, 555 + seed).reshape(int(cu[-1]), H, D)
    return spec, q, k, v, cu


def dense_causal(spec, q, k, v, cu, scale):
    """Matrix form per sequence and head: gather K,V dense, S = Q K^T, mask, softmax, P V."""
    H, D = q.shape[1], q.shape[2]
    G = H // spec.num_kv_heads
    out = np.zeros(q.shape, np.float64)
    qf = wl.bf16_bits_to_f64(q).astype(np.longdouble)
    for b in range(spec.batch):
        L, ql = int(spec.seq_lens[b]), int(cu[b + 1] - cu[b])
        if ql == 0:
            continue
        phys = spec.blocks_of(b)
        for h in range(H):
            K = wl.bf16_bits_to_f64(np.concatenate([k[p, h // G] for p in phys])[:L]).astype(np.longdouble)
            V = wl.bf16_bits_to_f64(np.concatenate([v[p, h // G] for p in phys])[:L]).astype(np.longdouble)
            S = (qf[cu[b]:cu[b + 1], h] @ K.T) * np.longdouble(scale)
            pos = L - ql + np.arange(ql)
            S = np.where(np.arange(L)[None, :] <= pos[:, None], S, -np.inf)
            P = np.exp(S - S.max(axis=1, keepdims=True))
            out[cu[b]:cu[b + 1], h] = ((P @ V) / P.sum(axis=1, keepdims=True)).astype(np.float64)
    return out


def test_matches_dense_causal_bruteforce():
    spec, q, k, v, cu = make_case([37, 64, 5, 130], [37, 10, 0, 33], H=4, Hkv=2)
    out = oracle.pa_prefill(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    ref = dense_causal(spec, q, k, v, cu, spec.scale)
    assert np.isfinite(out).all() and np.abs(out - ref).max() < 1e-12


def test_each_query_equals_a_decode_step_at_its_position():
    spec, q, k, v, cu = make_case([50, 21], [7, 21], H=6, Hkv=3, D=128, seed=2)
    out = oracle.pa_prefill(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    for b in range(2):
        ql = int(cu[b + 1] - cu[b])
        for i in range(ql):
            pos = int(spec.seq_lens[b]) - ql + i
            dec = oracle.pa_decode(q[cu[b] + i][None], k, v, spec.block_tables[b:b + 1],
                                   np.array([pos + 1], np.int32), spec.scale)
            assert (dec[0] == out[cu[b] + i]).all()


def test_chunked_prefill_equals_one_shot():
    # a 100-token prompt processed whole, or as chunks of 32 with growing context
    spec, q, k, v, cu = make_case([100], [100], H=2, Hkv=1, seed=3)
    whole = oracle.pa_prefill(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    for start in range(0, 100, 32):
        end = min(100, start + 32)
        part = oracle.pa_prefill(q[start:end], k, v, spec.block_tables, np.array([end], np.int32),
                                 np.array([0, end - start], np.int32), spec.scale)
        assert (part == whole[start:end]).all()


def test_first_token_attends_only_to_itself_and_poison_is_ignored():
    spec, q, k, v, cu = make_case([19], [19], H=2, Hkv=2, seed=4)      # tail slots are NaN
    out = oracle.pa_prefill(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    p = int(spec.block_tables[0, 0])
    assert (out[0] == wl.bf16_bits_to_f64(v[p, :, 0, :])).all()
    assert np.isfinite(out).all()


def test_invalid_lengths_refused():
    spec, q, k, v, cu = make_case([20, 8], [5, 8])
    with pytest.raises(ValueError):
        oracle.pa_prefill(q, k, v, spec.block_tables, np.array([4, 8], np.int32), cu, spec.scale)


@pytest.mark.parametrize("kind", ["no_mask", "offset", "strict"])
def test_bruteforce_catches_planted_causal_mistakes(kind):
    spec, q, k, v, cu = make_case([48], [20], H=2, Hkv=1, seed=5)
    ref = dense_causal(spec, q, k, v, cu, spec.scale)
    if kind == "no_mask":       # every query sees the whole context
        bad = np.stack([oracle.pa_decode(q[i][None], k, v, spec.block_tables, spec.seq_lens,
                                         spec.scale)[0] for i in range(20)])
    elif kind == "offset":      # positions counted from 0 instead of ctx - q_len
        bad = oracle.pa_prefill(q, k, v, spec.block_tables, np.array([20], np.int32), cu, spec.scale)
    else:                       # strict inequality: token does not see itself
        bad = oracle.pa_prefill(q, k, v, spec.block_tables, np.array([47], np.int32), cu, spec.scale)
    assert np.abs(bad - ref).max() > 1e-3
