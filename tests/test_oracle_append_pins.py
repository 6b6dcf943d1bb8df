"""Pins of the append oracle: equality with numpy fancy indexing, untouched bytes, padding,
and that appending a token then decoding equals decoding the longer sequence."""
import numpy as np
import pytest

import oracle
from paper_2602_07878_b200 import workloads as wl


def test_append_is_a_scatter_of_rows():
    spec = wl.make_spec("t", seq_lens=[5, 16, 31], num_q_heads=4, num_kv_heads=2, head_dim=64,
                        num_blocks=8, seed=3)
    k, v = wl.pools_np(spec, poison_tails=False)
    k0, v0 = k.copy(), v.copy()
    kn = wl.normal_bf16_np(0, 3 * 2 * 64, 70).reshape(3, 2, 64)
    vn = wl.normal_bf16_np(0, 3 * 2 * 64, 71).reshape(3, 2, 64)
    # token index L of each sequence (its next free slot); sequence 1 needs a fresh block
    blocks = [int(spec.block_tables[0, 0]), int(spec.free_blocks[0]), int(spec.block_tables[2, 1])]
    offs = [5, 0, 15]
    slots = np.array([b * 16 + o for b, o in zip(blocks, offs)], np.int64)
    oracle.kv_append(k, v, kn, vn, slots)
    ek, ev = k0.copy(), v0.copy()
    ek[blocks, :, offs, :] = kn          # numpy's own scatter
    ev[blocks, :, offs, :] = vn
    assert (k == ek).all() and (v == ev).all()
    # padding entries write nothing
    k2, v2 = k0.copy(), v0.copy()
    oracle.kv_append(k2, v2, kn, vn, np.array([-1, -1, -1], np.int64))
    assert (k2 == k0).all() and (v2 == v0).all()
    with pytest.raises(ValueError):
        oracle.kv_append(k2, v2, kn, vn, np.array([0, 8 * 16, 1], np.int64))


def test_append_then_decode_equals_decoding_the_longer_sequence():
    spec = wl.make_spec("t", seq_lens=[47, 16], num_q_heads=4, num_kv_heads=2, head_dim=64,
                        num_blocks=8, seed=4)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec, poison_tails=False)
    longer = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    # cut the last token of sequence 0 out, poison its slot, append it back
    p, j = int(spec.block_tables[0, 46 // 16]), 46 % 16
    kn, vn = k[p, :, j, :].copy()[None], v[p, :, j, :].copy()[None]
    k[p, :, j, :] = wl.BF16_NAN_BITS
    v[p, :, j, :] = wl.BF16_NAN_BITS
    lens = spec.seq_lens.copy()
    lens[0] = 46
    shorter = oracle.pa_decode(q, k, v, spec.block_tables, lens, spec.scale)
    assert np.isfinite(shorter).all() and np.abs(shorter[0] - longer[0]).max() > 1e-6
    oracle.kv_append(k, v, kn, vn, np.array([p * 16 + j], np.int64))
    again = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert (again == longer).all()
