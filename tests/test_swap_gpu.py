"""GPU swaps (through the C-ABI) are bit-exact against the swap oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from helpers import GpuDecode, bits_to_torch

pytestmark = pytest.mark.gpu


def make_pools(layers, NB, Hkv, D, seed=50):
    n = layers * NB * Hkv * 16 * D
    k = wl.normal_bf16_np(0, n, seed).reshape(layers, NB, Hkv, 16, D)
    v = wl.normal_bf16_np(0, n, seed + 1).reshape(layers, NB, Hkv, 16, D)
    return k, v


def as_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("staged", [False, True])
@pytest.mark.parametrize("layers,NB,Hkv,D", [(1, 40, 8, 64), (3, 64, 2, 128), (32, 24, 8, 128), (2, 30, 8, 256)])
def test_swap_out_and_in_bit_exact(staged, layers, NB, Hkv, D):
    k, v = make_pools(layers, NB, Hkv, D)
    kd, vd = bits_to_torch(k), bits_to_torch(v)
    rng = np.random.default_rng(layers)
    src = rng.permutation(NB)[:7].astype(np.int32)
    dst = rng.permutation(NB)[:7].astype(np.int32)
    bb = api.kv_block_bytes(kd, vd)
    assert bb == layers * 2 * Hkv * 16 * D * 2
    host = torch.zeros(7 * bb, dtype=torch.uint8).pin_memory()
    staging = torch.empty(3 * bb + 100, dtype=torch.uint8, device="cuda") if staged else None
    api.kv_swap_out(kd, vd, src, host, staging)
    torch.cuda.synchronize()
    expect = oracle.swap_out(k, v, src)
    assert (host.numpy().view(np.uint16) == expect.reshape(-1)).all()
    assert (as_bits(kd) == k).all() and (as_bits(vd) == v).all()      # source untouched
    api.kv_swap_in(kd, vd, host, dst, staging)
    torch.cuda.synchronize()
    k2, v2 = k.copy(), v.copy()
    oracle.swap_in(k2, v2, expect, dst)
    assert (as_bits(kd) == k2).all() and (as_bits(vd) == v2).all()    # every other byte unchanged


def test_swap_with_token_major_layout():
    layers, NB, Hkv, D = 2, 20, 4, 128
    k, v = make_pools(layers, NB, Hkv, D)
    kd = bits_to_torch(k).permute(0, 1, 3, 2, 4).contiguous().permute(0, 1, 3, 2, 4)
    vd = bits_to_torch(v).permute(0, 1, 3, 2, 4).contiguous().permute(0, 1, 3, 2, 4)
    ids = np.array([3, 19, 0], np.int32)
    host = torch.zeros(3 * api.kv_block_bytes(kd, vd), dtype=torch.uint8).pin_memory()
    api.kv_swap_out(kd, vd, ids, host)
    torch.cuda.synchronize()
    assert (host.numpy().view(np.uint16) == oracle.swap_out(k, v, ids).reshape(-1)).all()


def test_more_blocks_than_one_launch_carries():
    layers, NB, Hkv, D = 1, 1400, 1, 64
    k, v = make_pools(layers, NB, Hkv, D)
    kd, vd = bits_to_torch(k), bits_to_torch(v)
    ids = np.random.default_rng(2).permutation(NB)[:1100].astype(np.int32)
    host = torch.zeros(1100 * api.kv_block_bytes(kd, vd), dtype=torch.uint8).pin_memory()
    api.kv_swap_out(kd, vd, ids, host)
    torch.cuda.synchronize()
    assert (host.numpy().view(np.uint16) == oracle.swap_out(k, v, ids).reshape(-1)).all()


def test_unpinned_host_buffer_is_refused_in_direct_mode():
    k, v = make_pools(1, 8, 1, 64)
    kd, vd = bits_to_torch(k), bits_to_torch(v)
    host = torch.zeros(2 * api.kv_block_bytes(kd, vd), dtype=torch.uint8)   # pageable
    with pytest.raises(api.PagedKVError) as e:
        api.kv_swap_out(kd, vd, [1, 2], host)
    assert e.value.code == api.ERR["HOSTBUF"]


def test_cfg1_eviction_round_trip_keeps_decode_bits():
    """Workload 1: evict sequence 2 (100 tokens, 7 blocks), let its old blocks be
    overwritten, restore into 7 of the 11 free blocks, remap: decode output is unchanged."""
    spec = wl.config_spec(1)
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec)
    g = GpuDecode(spec, q, k, v)
    before = g.run().clone()
    src, dst = spec.blocks_of(2), spec.free_blocks[:7]
    kp, vp = g.k.unsqueeze(0), g.v.unsqueeze(0)
    host = torch.zeros(7 * api.kv_block_bytes(kp, vp), dtype=torch.uint8).pin_memory()
    api.kv_swap_out(kp, vp, src, host)
    torch.cuda.synchronize()
    expect = oracle.swap_out(k[None], v[None], src)
    assert (host.numpy().view(np.uint16) == expect.reshape(-1)).all()
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16, device="cuda")
    g.k[torch.from_numpy(src).long().cuda()] = nan
    g.v[torch.from_numpy(src).long().cuda()] = nan
    api.kv_swap_in(kp, vp, host, dst)
    t = spec.block_tables.copy()
    t[2, :7] = dst
    g.tables.copy_(torch.from_numpy(t))
    after = g.run()
    assert torch.equal(after.view(torch.int16), before.view(torch.int16))


@pytest.mark.parametrize("staged", [False, True])
def test_block_major_pool_swap_and_per_layer_decode(staged):
    # all layers of a block stored together ([NB][layer][K|V][Hkv][16][D]): the pools handed to
    # the library are strided views; swaps stay bit-exact, every other byte (the other blocks
    # of the interleaved store) stays untouched, and decode on one layer's view matches the
    # oracle with a block stride of layers * 2 * 32 KiB
    layers, NB, Hkv, D, H = 3, 48, 2, 128, 8
    k, v = make_pools(layers, NB, Hkv, D, seed=77)
    store = torch.empty(NB, layers, 2, Hkv, 16, D, dtype=torch.bfloat16, device="cuda")
    store[:, :, 0] = bits_to_torch(k).permute(1, 0, 2, 3, 4)
    store[:, :, 1] = bits_to_torch(v).permute(1, 0, 2, 3, 4)
    kd, vd = store[:, :, 0].permute(1, 0, 2, 3, 4), store[:, :, 1].permute(1, 0, 2, 3, 4)
    assert kd.stride(1) == layers * 2 * Hkv * 16 * D and not kd.is_contiguous()
    rng = np.random.default_rng(7)
    perm = rng.permutation(NB)
    src, dst = perm[:9].astype(np.int32), perm[9:18].astype(np.int32)
    bb = api.kv_block_bytes(kd, vd)
    host = torch.zeros(9 * bb, dtype=torch.uint8).pin_memory()
    staging = torch.empty(4 * bb, dtype=torch.uint8, device="cuda") if staged else None
    api.kv_swap_out(kd, vd, src, host, staging)
    torch.cuda.synchronize()
    image = oracle.swap_out(k, v, src)
    assert (host.numpy().view(np.uint16) == image.reshape(-1)).all()
    # in this layout a block's image is the block's own bytes
    assert (as_bits(store[int(src[0])]).reshape(-1) == image.reshape(9, -1)[0]).all()
    api.kv_swap_in(kd, vd, host, dst, staging)
    torch.cuda.synchronize()
    k2, v2 = k.copy(), v.copy()
    oracle.swap_in(k2, v2, image, dst)
    assert (as_bits(kd) == k2).all() and (as_bits(vd) == v2).all()
    # decode over layer 1 of the restored pool, tables pointing at the new ids
    lens = np.array([9 * 16 - 5, 40], np.int32)
    tables = np.full((2, 9), -1, np.int32)
    tables[0] = dst
    tables[1, :3] = perm[20:23]
    q = wl.normal_bf16_np(0, 2 * H * D, 78).reshape(2, H, D)
    qd = bits_to_torch(q)
    out = torch.empty_like(qd)
    shape = api.shape_of(kd[1], H)
    ws = torch.empty(api.pa_workspace_bytes(shape, 2, 16 * tables.size), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.pa_decode(qd, kd[1], vd[1], torch.from_numpy(tables).cuda(), torch.from_numpy(lens).cuda(),
                  D ** -0.5, out, ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.pa_decode(q, k2[1], v2[1], tables, lens, np.float32(D ** -0.5))
    from helpers import assert_parity, torch_to_f64
    assert_parity(torch_to_f64(out), ref, "block-major layer view")
