"""KV-head sharding on CPU: the head arithmetic, that per-rank results concatenate to the
definition (the oracle stands in for the kernels), and the same over two gloo ranks."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import oracle
from paper_2602_07878_b200 import kvshard
from paper_2602_07878_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def small_spec(seed=5):
    return wl.make_spec("t", seq_lens=[1, 15, 16, 17, 100, 0, 333], num_q_heads=16,
                        num_kv_heads=8, head_dim=64, occupancy=0.8, seed=seed)


@pytest.mark.parametrize("world", [1, 2, 4, 8])
def test_head_ranges_partition_the_heads_and_keep_groups_together(world):
    H, Hkv = 32, 8
    g = H // Hkv
    seen_q, seen_kv = [], []
    for r in range(world):
        qs, ks = kvshard.head_range(r, world, H, Hkv)
        seen_q += list(range(H))[qs]
        seen_kv += list(range(Hkv))[ks]
        # every query head of the slice reads a KV head of the slice, at the same local offset
        for i, h in enumerate(range(H)[qs]):
            assert h // g == ks.start + i // g
    assert seen_q == list(range(H)) and seen_kv == list(range(Hkv))


def test_bad_groups_are_refused():
    with pytest.raises(ValueError):
        kvshard.head_range(0, 3, 32, 8)     # 3 ranks do not divide 8 KV heads
    with pytest.raises(ValueError):
        kvshard.head_range(2, 2, 32, 8)
    with pytest.raises(ValueError):
        kvshard.head_range(0, 2, 12, 8)


def _oracle_decode_fn(q, k, v, tables, lens, scale, out, workspace, **kw):
    # strided views of uint16 bit patterns; the oracle takes the cache strides as they are
    ref = oracle.pa_decode(np.ascontiguousarray(q.numpy()), k.numpy(), v.numpy(), tables.numpy(),
                           lens.numpy(), scale)
    out.copy_(torch.from_numpy(ref))


@pytest.mark.parametrize("world", [1, 2, 4, 8])
def test_per_rank_results_concatenate_to_the_definition(world):
    spec = small_spec()
    k, v = wl.pools_np(spec)
    q = wl.q_np(spec)
    ref = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    out = torch.full(q.shape, float("nan"), dtype=torch.float64)
    for r in range(world):
        kvshard.decode(r, world, torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v),
                       torch.from_numpy(spec.block_tables), torch.from_numpy(spec.seq_lens),
                       spec.scale, out, None, decode_fn=_oracle_decode_fn)
    assert (out.numpy() == ref).all()       # rows are independent: exactly the same numbers


def test_swap_images_of_the_ranks_interleave_to_the_full_image():
    # a rank's image of a block is its heads' part of the full image, layer by layer
    layers, NB, Hkv, D = 3, 10, 4, 64
    n = layers * NB * Hkv * 16 * D
    k = wl.normal_bf16_np(0, n, 41).reshape(layers, NB, Hkv, 16, D)
    v = wl.normal_bf16_np(0, n, 42).reshape(layers, NB, Hkv, 16, D)
    ids = np.array([7, 2, 9], np.int32)
    full = oracle.swap_out(k, v, ids)                       # [n, layers, 2, Hkv, 16, D]
    for world in (2, 4):
        for r in range(world):
            _, ks = kvshard.head_range(r, world, Hkv, Hkv)
            img = oracle.swap_out(k[:, :, ks], v[:, :, ks], ids)
            assert (img == full[:, :, :, ks]).all()


def _worker(rank, world, port, q_out):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank,
                            world_size=world)
    spec = small_spec(seed=12)
    k, v = wl.pools_np(spec)
    q = wl.q_np(spec)
    out = torch.zeros(q.shape, dtype=torch.float64)
    mine = kvshard.decode(rank, world, torch.from_numpy(q), torch.from_numpy(k),
                          torch.from_numpy(v), torch.from_numpy(spec.block_tables),
                          torch.from_numpy(spec.seq_lens), spec.scale, out, None,
                          decode_fn=_oracle_decode_fn)
    # outside the path: what a tensor-parallel layer would do next needs every head somewhere;
    # here the slices are simply gathered so that the test can look at the whole result
    pieces = [torch.zeros_like(mine).contiguous() for _ in range(world)]
    dist.all_gather(pieces, mine.contiguous())
    dist.barrier()
    dist.destroy_process_group()
    q_out.put((rank, torch.cat(pieces, dim=1).numpy()))


def test_two_gloo_ranks_cover_all_heads():
    ctx = mp.get_context("spawn")
    qu = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29641, qu)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((qu.get(timeout=180) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    spec = small_spec(seed=12)
    k, v = wl.pools_np(spec)
    ref = oracle.pa_decode(wl.q_np(spec), k, v, spec.block_tables, spec.seq_lens, spec.scale)
    for _, out in res:
        assert (out == ref).all()
