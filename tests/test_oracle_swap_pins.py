"""Pins of the swap oracle: the host image is the plain concatenation of block payloads
(checked against numpy fancy indexing), swap-in touches nothing else, and a round trip
through different block ids preserves the decode oracle's output."""
import numpy as np
import pytest

import oracle
from paper_2602_07878_b200 import workloads as wl


def _pools(layers=3, NB=12, Hkv=2, bs=16, D=64, seed=77):
    n = layers * NB * Hkv * bs * D
    k = wl.normal_bf16_np(0, n, seed).reshape(layers, NB, Hkv, bs, D)
    v = wl.normal_bf16_np(0, n, seed + 1).reshape(layers, NB, Hkv, bs, D)
    return k, v


def test_swap_out_is_block_concatenation():
    k, v = _pools()
    ids = np.array([7, 0, 11, 3], np.int32)
    host = oracle.swap_out(k, v, ids)
    assert host.shape == (4, 3, 2, 2, 16, 64)
    # numpy definition: host[i, l, 0] = K[l, ids[i]], host[i, l, 1] = V[l, ids[i]]
    assert (host[:, :, 0] == k[:, ids].transpose(1, 0, 2, 3, 4)).all()
    assert (host[:, :, 1] == v[:, ids].transpose(1, 0, 2, 3, 4)).all()


def test_swap_out_respects_strides():
    k, v = _pools()
    # same logical content stored [layers, NB, bs, Hkv, D]
    k2 = np.ascontiguousarray(k.transpose(0, 1, 3, 2, 4)).transpose(0, 1, 3, 2, 4)
    v2 = np.ascontiguousarray(v.transpose(0, 1, 3, 2, 4)).transpose(0, 1, 3, 2, 4)
    ids = np.array([5, 2], np.int32)
    assert (oracle.swap_out(k, v, ids) == oracle.swap_out(k2, v2, ids)).all()


def test_swap_in_writes_only_the_listed_blocks():
    k, v = _pools()
    k0, v0 = k.copy(), v.copy()
    src = np.array([1, 4, 9], np.int32)
    dst = np.array([10, 2, 6], np.int32)
    host = oracle.swap_out(k, v, src)
    oracle.swap_in(k, v, host, dst)
    others = np.setdiff1d(np.arange(12), dst)
    assert (k[:, others] == k0[:, others]).all() and (v[:, others] == v0[:, others]).all()
    assert (k[:, dst] == k0[:, src]).all() and (v[:, dst] == v0[:, src]).all()
    # reading the same ids back returns the identical image
    assert (oracle.swap_out(k, v, dst) == host).all()


def test_swap_bad_id_is_refused():
    k, v = _pools()
    with pytest.raises(ValueError):
        oracle.swap_out(k, v, np.array([12], np.int32))
    with pytest.raises(ValueError):
        oracle.swap_in(k, v, np.zeros((1, 3, 2, 2, 16, 64), np.uint16), np.array([-1], np.int32))


def test_cfg1_round_trip_keeps_decode_output():
    # evict the 100-token sequence (index 2, 7 blocks, partial last block), restore it into
    # 7 of the 11 free blocks, remap its table row: the attention output must not move
    spec = wl.config_spec(1)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    before = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    src = spec.blocks_of(2)
    assert len(src) == 7 and len(spec.free_blocks) == 11
    dst = spec.free_blocks[:7]
    k5, v5 = k[None].copy(), v[None].copy()
    host = oracle.swap_out(k5, v5, src)
    k5[0, src] = wl.BF16_NAN_BITS           # the freed blocks may be overwritten by anyone
    v5[0, src] = wl.BF16_NAN_BITS
    oracle.swap_in(k5, v5, host, dst)
    t = spec.block_tables.copy()
    t[2, :7] = dst
    after = oracle.pa_decode(q, k5[0], v5[0], t, spec.seq_lens, spec.scale)
    assert (after == before).all()
