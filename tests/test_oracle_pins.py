"""Pins of the fp64 decode oracle against things other than itself (CPU only).

The paper prints no worked numerical example of attention, so the pins are: brute-force
dense attention on un-paged copies (long double, no max subtraction, separately written),
closed forms, invariants, and checks that a planted mistake is caught.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2602_07878_b200 import workloads as wl


def dense_bruteforce(q_bits, k_bits, v_bits, tables, lens, scale):
    """softmax(q K^T scale) V with K/V first gathered to dense [L, D]; long double,
    plain sum(exp(s) v) / sum(exp(s)) without subtracting the maximum."""
    B, H, D = q_bits.shape
    NB, Hkv, bs, _ = k_bits.shape
    G = H // Hkv
    q = wl.bf16_bits_to_f64(q_bits).astype(np.longdouble)
    out = np.zeros((B, H, D), dtype=np.longdouble)
    for b in range(B):
        L = int(lens[b])
        if L == 0:
            continue
        nb = (L + bs - 1) // bs
        phys = [int(x) for x in tables[b, :nb]]
        for h in range(H):
            kvh = h // G
            Kd = np.concatenate([k_bits[p, kvh] for p in phys], axis=0)[:L]
            Vd = np.concatenate([v_bits[p, kvh] for p in phys], axis=0)[:L]
            Kd = wl.bf16_bits_to_f64(Kd).astype(np.longdouble)
            Vd = wl.bf16_bits_to_f64(Vd).astype(np.longdouble)
            e = np.exp((Kd @ q[b, h]) * np.longdouble(scale))
            out[b, h] = (e[:, None] * Vd).sum(axis=0) / e.sum()
    return out.astype(np.float64)


def run_spec(spec, poison=True, **kw):
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec, poison_tails=poison)
    out = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale, **kw)
    return q, k, v, out


def test_bruteforce_dense_cfg1():
    spec = wl.config_spec(1)
    q, k, v, out = run_spec(spec)
    ref = dense_bruteforce(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() < 1e-12


@pytest.mark.parametrize("H,Hkv,D", [(4, 4, 64), (8, 2, 128), (8, 1, 32), (6, 3, 128)])
def test_bruteforce_dense_gqa_shapes(H, Hkv, D):
    spec = wl.make_spec("t", seq_lens=[1, 15, 16, 17, 33, 0, 70], num_q_heads=H,
                        num_kv_heads=Hkv, head_dim=D, num_blocks=24, seed=H * 100 + D)
    q, k, v, out = run_spec(spec)
    ref = dense_bruteforce(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert np.abs(out - ref).max() < 1e-12
    assert (out[5] == 0).all()            # L = 0 row is zeros


def test_strided_pool_layout_matches_dense():
    # pool stored [NB, bs, Hkv, D] and viewed as [NB, Hkv, bs, D]: strides, not layout, decide
    spec = wl.make_spec("t", seq_lens=[40, 9], num_q_heads=4, num_kv_heads=2, head_dim=64,
                        num_blocks=8, seed=11)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    k2 = np.ascontiguousarray(k.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)
    v2 = np.ascontiguousarray(v.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)
    assert not k2.flags["C_CONTIGUOUS"]
    a = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    b = oracle.pa_decode(q, k2, v2, spec.block_tables, spec.seq_lens, spec.scale)
    assert (a == b).all()


def test_physical_permutation_invariance():
    spec = wl.config_spec(1)
    q, k, v, out = run_spec(spec)
    rng = np.random.default_rng(3)
    perm = rng.permutation(spec.num_blocks)          # new id of old block p is perm[p]
    k2 = np.empty_like(k)
    v2 = np.empty_like(v)
    k2[perm] = k
    v2[perm] = v
    t2 = spec.block_tables.copy()
    for b in range(spec.batch):
        nb = len(spec.blocks_of(b))
        t2[b, :nb] = perm[spec.block_tables[b, :nb]]
    out2 = oracle.pa_decode(q, k2, v2, t2, spec.seq_lens, spec.scale)
    assert (out == out2).all()


def test_batch_composition_invariance():
    spec = wl.config_spec(1)
    q, k, v, out = run_spec(spec)
    order = [2, 0, 3, 1]
    out_p = oracle.pa_decode(q[order], k, v, spec.block_tables[order], spec.seq_lens[order],
                             spec.scale)
    assert (out_p == out[order]).all()
    for b in range(spec.batch):
        alone = oracle.pa_decode(q[b:b + 1], k, v, spec.block_tables[b:b + 1],
                                 spec.seq_lens[b:b + 1], spec.scale)
        assert (alone[0] == out[b]).all()


def test_thread_count_does_not_change_result():
    spec = wl.config_spec(1)
    _, _, _, a = run_spec(spec, num_threads=1)
    _, _, _, b = run_spec(spec, num_threads=0)
    assert (a == b).all()


def test_equal_keys_give_mean_of_values():
    spec = wl.make_spec("t", seq_lens=[37, 64], num_q_heads=4, num_kv_heads=2, head_dim=64,
                        num_blocks=10, seed=5)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    krow = wl.normal_bf16_np(0, 64, 999)
    k[:, :, :, :] = krow                    # every key identical (tails included)
    out = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    vf = wl.bf16_bits_to_f64(v)
    for b in range(2):
        L = int(spec.seq_lens[b])
        for h in range(4):
            rows = np.concatenate([vf[p, h // 2] for p in spec.blocks_of(b)])[:L]
            assert np.abs(out[b, h] - rows.mean(axis=0)).max() < 1e-13


def test_zero_scale_and_zero_query_give_mean():
    spec = wl.make_spec("t", seq_lens=[50], num_q_heads=2, num_kv_heads=2, head_dim=64,
                        num_blocks=5, seed=6)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    vf = wl.bf16_bits_to_f64(v)
    mean = [np.concatenate([vf[p, h] for p in spec.blocks_of(0)])[:50].mean(axis=0)
            for h in range(2)]
    a = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, 0.0)
    b = oracle.pa_decode(np.zeros_like(q), k, v, spec.block_tables, spec.seq_lens, spec.scale)
    for h in range(2):
        assert np.abs(a[0, h] - mean[h]).max() < 1e-13
        assert np.abs(b[0, h] - mean[h]).max() < 1e-13


def test_single_token_returns_its_value_exactly():
    spec = wl.make_spec("t", seq_lens=[1, 1], num_q_heads=4, num_kv_heads=4, head_dim=128,
                        num_blocks=4, seed=7)
    q, k, v, out = run_spec(spec)
    vf = wl.bf16_bits_to_f64(v)
    for b in range(2):
        p = int(spec.block_tables[b, 0])
        assert (out[b] == vf[p, :, 0, :]).all()


def test_two_tokens_logistic_weights():
    # D = 2, q = (1, 0): s_t = scale * K_t[0]; weights are logistic in s_0 - s_1
    D = 2
    q = wl.f64_to_bf16_bits(np.array([[[1.0, 0.0]]]))
    k = np.zeros((1, 1, 16, D), dtype=np.uint16)
    v = np.zeros((1, 1, 16, D), dtype=np.uint16)
    k[0, 0, 0] = wl.f64_to_bf16_bits(np.array([0.5, 3.0]))
    k[0, 0, 1] = wl.f64_to_bf16_bits(np.array([-1.25, -7.0]))
    v[0, 0, 0] = wl.f64_to_bf16_bits(np.array([1.0, -2.0]))
    v[0, 0, 1] = wl.f64_to_bf16_bits(np.array([3.0, 4.0]))
    k[0, 0, 2:] = wl.BF16_NAN_BITS
    v[0, 0, 2:] = wl.BF16_NAN_BITS
    scale = 2.0
    out = oracle.pa_decode(q, k, v, np.array([[0]], np.int32), np.array([2], np.int32), scale)
    w0 = 1.0 / (1.0 + math.exp(-scale * (0.5 + 1.25)))
    expect = w0 * np.array([1.0, -2.0]) + (1 - w0) * np.array([3.0, 4.0])
    assert np.abs(out[0, 0] - expect).max() < 1e-15


def test_dominant_key_selects_its_value():
    spec = wl.make_spec("t", seq_lens=[90], num_q_heads=1, num_kv_heads=1, head_dim=64,
                        num_blocks=6, seed=8)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    qf = wl.bf16_bits_to_f64(q[0, 0])
    # token 41 gets key = 64 * q / |q|^2-ish so that its score towers over N(0,1) scores
    big = wl.f64_to_bf16_bits(qf * 16.0)
    p, j = int(spec.block_tables[0, 41 // 16]), 41 % 16
    k[p, 0, j] = big
    out = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, 1.0)
    s_big = float(wl.bf16_bits_to_f64(big) @ qf)
    assert s_big > 400
    assert np.abs(out[0, 0] - wl.bf16_bits_to_f64(v[p, 0, j])).max() < 1e-15


def test_score_shift_invariance_and_large_scores():
    # q = (x, 1, 0...): adding c to component 1 of every key adds c*scale to every score
    D = 64
    rng = np.random.default_rng(9)
    spec = wl.make_spec("t", seq_lens=[45], num_q_heads=1, num_kv_heads=1, head_dim=D,
                        num_blocks=3, seed=9)
    q = wl.q_np(spec)
    q[0, 0, 1] = wl.f64_to_bf16_bits(np.array(1.0))
    k, v = wl.pools_np(spec, poison_tails=False)
    k[..., 1] = wl.f64_to_bf16_bits(rng.integers(-4, 4, size=k.shape[:-1]) * 0.5)
    base = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, 1.0)
    for c in (16.0, -24.0, 96.0):            # exact in bf16 together with multiples of 0.5
        k2 = k.copy()
        k2[..., 1] = wl.f64_to_bf16_bits(wl.bf16_bits_to_f64(k[..., 1]) + c)
        assert (wl.bf16_bits_to_f64(k2[..., 1]) == wl.bf16_bits_to_f64(k[..., 1]) + c).all()
        shifted = oracle.pa_decode(q, k2, v, spec.block_tables, spec.seq_lens, 1.0)
        assert np.isfinite(shifted).all()
        assert np.abs(shifted - base).max() < 1e-12


def test_gqa_equals_mha_with_replicated_kv_heads():
    spec = wl.make_spec("t", seq_lens=[33, 100], num_q_heads=8, num_kv_heads=2, head_dim=64,
                        num_blocks=12, seed=10)
    q, k, v, out = run_spec(spec)
    k_rep = np.repeat(k, 4, axis=1)
    v_rep = np.repeat(v, 4, axis=1)
    out_mha = oracle.pa_decode(q, k_rep, v_rep, spec.block_tables, spec.seq_lens, spec.scale)
    assert (out == out_mha).all()
    # head h reads KV head h // 4 only
    k2 = k.copy()
    k2[:, 1] = wl.normal_bf16_np(0, k[:, 1].size, 4242).reshape(k[:, 1].shape)
    out2 = oracle.pa_decode(q, k2, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert (out2[:, :4] == out[:, :4]).all()
    assert not (out2[:, 4:] == out[:, 4:]).all()


def test_unused_slots_and_table_entries_are_never_read():
    spec = wl.config_spec(1)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec, poison_tails=False)
    clean = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    kp, vp = wl.pools_np(spec, poison_tails=True)
    assert (kp != k).any()
    t = spec.block_tables.copy()
    assert (t == -1).any() and (t == 0x7FFFFFFF).any()
    poisoned = oracle.pa_decode(q, kp, vp, t, spec.seq_lens, spec.scale)
    assert np.isfinite(poisoned).all() and (poisoned == clean).all()
    # unreferenced physical blocks do not matter either
    for p in spec.free_blocks:
        kp[p] = wl.BF16_NAN_BITS
        vp[p] = wl.BF16_NAN_BITS
    assert (oracle.pa_decode(q, kp, vp, t, spec.seq_lens, spec.scale) == clean).all()


def test_shared_prefix_block_is_legal():
    spec = wl.make_spec("t", seq_lens=[40, 40], num_q_heads=2, num_kv_heads=2, head_dim=64,
                        num_blocks=8, seed=12)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    t = spec.block_tables.copy()
    t[1, 0] = t[0, 0]                      # both sequences share their first block
    out = oracle.pa_decode(q, k, v, t, spec.seq_lens, spec.scale)
    ref = dense_bruteforce(q, k, v, t, spec.seq_lens, spec.scale)
    assert np.abs(out - ref).max() < 1e-12


def test_duplicated_context_leaves_output_unchanged():
    # L -> 2L with the same tokens twice: softmax weights halve, the mixture is the same
    spec = wl.make_spec("t", seq_lens=[48], num_q_heads=2, num_kv_heads=1, head_dim=64,
                        num_blocks=8, seed=13)
    q, k, v, out = run_spec(spec)
    t2 = np.concatenate([spec.block_tables[:, :3], spec.block_tables[:, :3]], axis=1)
    out2 = oracle.pa_decode(q, k, v, t2, np.array([96], np.int32), spec.scale)
    assert np.abs(out2 - out).max() < 1e-14


def test_invalid_inputs_are_refused():
    spec = wl.config_spec(1)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    t = spec.block_tables.copy()
    t[0, 0] = spec.num_blocks
    with pytest.raises(ValueError):
        oracle.pa_decode(q, k, v, t, spec.seq_lens, spec.scale)
    lens = spec.seq_lens.copy()
    lens[3] = spec.max_blocks * 16 + 1
    with pytest.raises(ValueError):
        oracle.pa_decode(q, k, v, spec.block_tables, lens, spec.scale)


# --- planted mistakes: each pin above must be able to see a plausible bug -----------------
def _mutants():
    def wrong_head_map(q, k, v, t, lens, scale):       # kvh = h % Hkv instead of h // G
        H, Hkv = q.shape[1], k.shape[1]
        idx = [(h % Hkv) for h in range(H)]
        return oracle.pa_decode(q, k[:, idx], v[:, idx], t, lens, scale)

    def off_by_one_len(q, k, v, t, lens, scale):        # reads one token too few
        return oracle.pa_decode(q, k, v, t, np.maximum(lens - 1, 1), scale)

    def swapped_kv(q, k, v, t, lens, scale):            # K and V exchanged
        return oracle.pa_decode(q, v, k, t, lens, scale)

    def identity_table(q, k, v, t, lens, scale):        # ignores the logical->physical map
        t2 = np.tile(np.arange(t.shape[1], dtype=np.int32), (t.shape[0], 1))
        return oracle.pa_decode(q, k, v, t2, lens, scale)

    def no_scale(q, k, v, t, lens, scale):
        return oracle.pa_decode(q, k, v, t, lens, 1.0)

    return [wrong_head_map, off_by_one_len, swapped_kv, identity_table, no_scale]


@pytest.mark.parametrize("mutant", _mutants(), ids=lambda f: f.__name__)
def test_bruteforce_pin_catches_planted_mistakes(mutant):
    spec = wl.make_spec("t", seq_lens=[17, 64, 35], num_q_heads=8, num_kv_heads=4,
                        head_dim=64, num_blocks=12, seed=14)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec, poison_tails=False)
    ref = dense_bruteforce(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    bad = mutant(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert np.abs(bad - ref).max() > 1e-3


def test_scale_is_rounded_to_fp32_by_the_oracle_itself():
    # The scale is an fp32 argument of the method.  A Python double that is not an fp32 value
    # (0.1, 1/sqrt(128)) must give exactly what its fp32 rounding gives, and that must be the
    # brute-force result for the widened fp32 value -- not for the double.
    spec = wl.make_spec("t", seq_lens=[9, 40, 17], num_q_heads=4, num_kv_heads=2, head_dim=64,
                        num_blocks=12, seed=5)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    cu = np.array([0, 3, 10, 11], np.int32)
    qp = wl.normal_bf16_np(0, 11 * 4 * 64, 31).reshape(11, 4, 64)
    for s in (0.1, 128 ** -0.5, 3.3):
        s32 = np.float32(s)
        assert float(s32) != s
        a = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, s)
        assert (a == oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, s32)).all()
        ref32 = dense_bruteforce(q, k, v, spec.block_tables, spec.seq_lens, float(s32))
        ref64 = dense_bruteforce(q, k, v, spec.block_tables, spec.seq_lens, s)
        assert np.abs(a - ref32).max() < 1e-12
        assert np.abs(a - ref64).max() > np.abs(a - ref32).max()
        p = oracle.pa_prefill(qp, k, v, spec.block_tables, spec.seq_lens, cu, s)
        assert (p == oracle.pa_prefill(qp, k, v, spec.block_tables, spec.seq_lens, cu, s32)).all()
