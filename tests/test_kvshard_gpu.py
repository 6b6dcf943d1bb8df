"""KV-head sharding (tensor-parallel ranks) on one GPU: ranks run one after another on their
heads of batch-wide tensors -- strided views, nothing copied -- through the C-ABI.  No rank's
kernels wait on another's, so running them in sequence is the same computation."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api, kvshard
from paper_2602_07878_b200 import workloads as wl
from helpers import GpuDecode, assert_parity, bits_to_torch, oracle_for, torch_to_f64

pytestmark = pytest.mark.gpu


def as_bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("world", [2, 4, 8])
@pytest.mark.parametrize("H,Hkv,D", [(32, 8, 128), (8, 8, 64), (16, 8, 256)])
def test_sharded_decode_equals_unsharded_bits_and_the_oracle(world, H, Hkv, D):
    lens = [0, 5, 700, 16, 1300, 4100, 33, 512, 513]
    spec = wl.make_spec("t", seq_lens=lens, num_q_heads=H, num_kv_heads=Hkv, head_dim=D,
                        occupancy=0.9, seed=world * 100 + H)
    q, (k, v) = wl.q_np(spec), wl.pools_np(spec)
    ref = oracle_for(spec, q, k, v)
    P = 256   # a fixed partition size: a row's bits then depend on its own tokens only
    g = GpuDecode(spec, q, k, v, partition_tokens=P)
    whole = g.run().clone()
    assert_parity(torch_to_f64(whole), ref, "unsharded")
    out = torch.full_like(g.q, float("nan"))
    ws = torch.empty(kvshard.workspace_bytes(world, g.k, H, spec.batch, spec.total_tokens + 16 * 9, P),
                     dtype=torch.uint8, device="cuda")
    for r in range(world):
        out_r = kvshard.decode(r, world, g.q, g.k, g.v, g.tables, g.lens, spec.scale, out, ws,
                               partition_tokens=P, dev_status=g.status)
        if world > 1:
            assert not out_r.is_contiguous()     # the strided entry point took it
    torch.cuda.synchronize()
    assert int(g.status.item()) == 0
    assert torch.equal(out.view(torch.int16), whole.view(torch.int16))
    # the library's own choice of partition size depends on the rank's head count: same
    # definition, possibly another order of the fp32 sums
    out2 = torch.full_like(g.q, float("nan"))
    for r in range(world):
        kvshard.decode(r, world, g.q, g.k, g.v, g.tables, g.lens, spec.scale, out2, ws,
                       dev_status=g.status)
    torch.cuda.synchronize()
    assert_parity(torch_to_f64(out2), ref, f"world {world}, automatic partitions")
    # a rank that copies its slices instead gets the same bits as through the views
    qs, ks = kvshard.head_range(1, world, H, Hkv)
    qc, kc, vc = g.q[:, qs].contiguous(), g.k[:, ks].contiguous(), g.v[:, ks].contiguous()
    oc = torch.empty_like(qc)
    api.pa_decode(qc, kc, vc, g.tables, g.lens, spec.scale, oc, ws, partition_tokens=P)
    torch.cuda.synchronize()
    assert torch.equal(oc.view(torch.int16), whole[:, qs].contiguous().view(torch.int16))


def test_strided_views_leave_the_other_heads_alone_and_bad_strides_are_refused():
    spec = wl.make_spec("t", seq_lens=[40, 700, 0], num_q_heads=8, num_kv_heads=4, head_dim=128,
                        occupancy=0.9, seed=3)
    q, (k, v) = wl.q_np(spec), wl.pools_np(spec)
    g = GpuDecode(spec, q, k, v)
    # q as the first part of a wider per-token row (a fused projection), out likewise
    wide_q = torch.full((3, 8 * 128 + 2 * 4 * 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    wide_q[:, :1024] = g.q.reshape(3, -1)
    wide_o = torch.full((3, 1024 + 64), 7.0, dtype=torch.bfloat16, device="cuda")
    qv, ov = wide_q[:, :1024].view(3, 8, 128), wide_o[:, :1024].view(3, 8, 128)
    api.pa_decode(qv, g.k, g.v, g.tables, g.lens, spec.scale, ov, g.ws, dev_status=g.status)
    torch.cuda.synchronize()
    assert_parity(torch_to_f64(ov), oracle_for(spec, q, k, v), "q inside a wider row")
    assert bool((wide_o[:, 1024:] == 7.0).all())
    shape = api.shape_of(g.k, 8)
    import ctypes
    call = lambda qs, os_: api.lib().pa_decode_strided(
        ctypes.byref(shape), ctypes.c_void_p(g.q.data_ptr()), qs, ctypes.c_void_p(g.k.data_ptr()),
        ctypes.c_void_p(g.v.data_ptr()), ctypes.c_void_p(g.tables.data_ptr()), g.tables.shape[1],
        ctypes.c_void_p(g.lens.data_ptr()), 3, 0.1, ctypes.c_void_p(g.out.data_ptr()), os_,
        ctypes.c_void_p(g.ws.data_ptr()), g.ws.numel(), 0, 0, None, None)
    n0 = api.pa_launch_count()
    assert call(1024 - 8, 1024) == api.ERR["ARG"]        # rows of consecutive sequences overlap
    assert call(1024, 0) == api.ERR["ARG"]
    assert call(1024 + 4, 1024) == api.ERR["ALIGN"]      # rows would lose 16-byte alignment
    assert api.pa_launch_count() == n0


@pytest.mark.parametrize("world", [2, 4])
@pytest.mark.parametrize("staged", [False, True])
def test_sharded_swaps_are_bit_exact_and_touch_only_their_heads(world, staged):
    layers, NB, Hkv, D = 3, 40, 8, 128
    n = layers * NB * Hkv * 16 * D
    k = wl.normal_bf16_np(0, n, 61).reshape(layers, NB, Hkv, 16, D)
    v = wl.normal_bf16_np(0, n, 62).reshape(layers, NB, Hkv, 16, D)
    kd, vd = bits_to_torch(k), bits_to_torch(v)
    rng = np.random.default_rng(world)
    perm = rng.permutation(NB)
    src, dst = perm[:9].astype(np.int32), perm[9:18].astype(np.int32)
    k2, v2 = k.copy(), v.copy()
    for r in range(world):
        _, ks = kvshard.head_range(r, world, Hkv, Hkv)
        kr, vr = kd[:, :, ks], vd[:, :, ks]              # this rank's heads of the pools
        bb = api.kv_block_bytes(kr, vr)
        assert bb == layers * 2 * (Hkv // world) * 16 * D * 2
        host = torch.zeros(9 * bb, dtype=torch.uint8).pin_memory()
        staging = torch.empty(4 * bb, dtype=torch.uint8, device="cuda") if staged else None
        api.kv_swap_out(kr, vr, src, host, staging)
        torch.cuda.synchronize()
        image = oracle.swap_out(k[:, :, ks], v[:, :, ks], src)
        assert (host.numpy().view(np.uint16) == image.reshape(-1)).all()
        api.kv_swap_in(kr, vr, host, dst, staging)
        torch.cuda.synchronize()
        oracle.swap_in(k2[:, :, ks], v2[:, :, ks], image, dst)
        # heads of the ranks that have not swapped yet are still the original ones
        assert (as_bits(kd) == k2).all() and (as_bits(vd) == v2).all()
    full = oracle.swap_out(k, v, src)
    k3, v3 = k.copy(), v.copy()
    oracle.swap_in(k3, v3, full, dst)
    assert (k2 == k3).all() and (v2 == v3).all()         # all ranks together = the unsharded swap
