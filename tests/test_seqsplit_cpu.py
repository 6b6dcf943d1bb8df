"""Sequence-split decode on CPU: pins of the partial/merge oracle, the host-side sharding, and
the two-rank exchange over gloo with the oracle standing in for the kernels."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import oracle
from oracle import partials
from paper_2602_07878_b200 import seqsplit
from paper_2602_07878_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def small_spec(seed=3, lens=(1, 15, 16, 17, 100, 0, 333)):
    return wl.make_spec("t", seq_lens=list(lens), num_q_heads=4, num_kv_heads=2, head_dim=64,
                        occupancy=0.8, seed=seed)


# ---- pins of the oracle's partial / merge --------------------------------------------------
def test_merge_of_two_hand_made_parts_is_the_weighted_mean():
    # part A: m = 0, l = 1, o = (1, 0); part B: m = ln 3, l = 1, o = (0, 1):
    # weights e^0 : e^(ln 3) = 1 : 3 -> out = (1/4, 3/4)
    a = (np.array([[[1.0, 0.0]]]), np.array([[0.0]]), np.array([[1.0]]))
    b = (np.array([[[0.0, 1.0]]]), np.array([[np.log(3.0)]]), np.array([[1.0]]))
    out = partials.merge_partials([a, b])
    np.testing.assert_allclose(out[0, 0], [0.25, 0.75], rtol=0, atol=1e-15)
    # order of the parts does not matter, and a part's (o, l) may be scaled together with a
    # shift of its m: (o, m, l) == (o * e^c, m - c, l * e^c)
    c = 1.7
    b2 = (b[0] * np.exp(c), b[1] - c, b[2] * np.exp(c))
    np.testing.assert_allclose(partials.merge_partials([b2, a]), out, rtol=0, atol=1e-15)


def test_partial_of_one_token_is_that_value_row():
    spec = small_spec(lens=(1,))
    k, v = wl.pools_np(spec)
    q = wl.q_np(spec)
    o, m, l = partials.decode_partial(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    blk = spec.block_tables[0, 0]
    for h in range(4):
        np.testing.assert_array_equal(o[0, h], wl.bf16_bits_to_f64(v[blk, h // 2, 0]))
        assert l[0, h] == 1.0
        s = spec.scale * np.dot(wl.bf16_bits_to_f64(q[0, h]), wl.bf16_bits_to_f64(k[blk, h // 2, 0]))
        assert abs(m[0, h] - s) < 1e-12


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_merged_slices_equal_the_full_definition(world):
    spec = small_spec(seed=world)
    k, v = wl.pools_np(spec)
    q = wl.q_np(spec)
    ref = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    parts = []
    for r in range(world):
        t, ln = seqsplit.shard_context(spec.block_tables, spec.seq_lens, r, world)
        parts.append(partials.decode_partial(q, k, v, t, ln, spec.scale))
    out = partials.merge_partials(parts)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    assert (out[5] == 0).all()  # the empty sequence


def test_an_empty_part_has_weight_zero():
    spec = small_spec(lens=(40,))
    k, v = wl.pools_np(spec)
    q = wl.q_np(spec)
    full = partials.decode_partial(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    empty = partials.decode_partial(q, k, v, spec.block_tables, np.array([0], np.int32), spec.scale)
    assert np.isneginf(empty[1]).all() and (empty[2] == 0).all() and (empty[0] == 0).all()
    ref = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    np.testing.assert_allclose(partials.merge_partials([empty, full, empty]), ref, atol=1e-12)


# ---- host-side sharding ----------------------------------------------------------------------
@pytest.mark.parametrize("world", [1, 2, 4, 5])
def test_shards_partition_every_sequence(world):
    spec = small_spec(lens=(1, 16, 17, 31, 32, 33, 0, 1000, 77))
    seen = [[] for _ in range(spec.batch)]
    total = np.zeros(spec.batch, dtype=np.int64)
    for r in range(world):
        t, ln = seqsplit.shard_context(spec.block_tables, spec.seq_lens, r, world)
        assert t.dtype == np.int32 and ln.dtype == np.int32
        total += ln
        for b in range(spec.batch):
            nb = (int(ln[b]) + 15) // 16
            seen[b] += list(t[b, :nb])
            assert (t[b, nb:] == -1).all()
            # only the slice that holds the end of the sequence may end inside a block
            if ln[b] % 16:
                assert total[b] == spec.seq_lens[b]
    np.testing.assert_array_equal(total, spec.seq_lens)
    for b in range(spec.batch):
        nb = (int(spec.seq_lens[b]) + 15) // 16
        assert seen[b] == list(spec.block_tables[b, :nb])


def test_shard_rank_out_of_range():
    spec = small_spec()
    with pytest.raises(ValueError):
        seqsplit.shard_context(spec.block_tables, spec.seq_lens, 2, 2)


# ---- two gloo ranks: the exchange and the step's control flow ----------------------------------
def _oracle_partial_fn(q, k, v, tables, lens, scale, part, workspace, **kw):
    B, H, D = q.shape
    o, m, l = partials.decode_partial(q.numpy(), k.numpy(), v.numpy(), tables.numpy(),
                                      lens.numpy(), scale)
    rec = part.numpy()
    rec[: B * H * D] = o.reshape(-1)
    rec[B * H * D:] = np.stack([m, l], axis=-1).reshape(-1)


def _oracle_merge_fn(gathered, rows, D, out):
    g = gathered.numpy()
    parts = [(g[r, : rows * D].reshape(1, rows, D), g[r, rows * D:].reshape(1, rows, 2)[..., 0],
              g[r, rows * D:].reshape(1, rows, 2)[..., 1]) for r in range(g.shape[0])]
    out.copy_(torch.from_numpy(partials.merge_partials(parts).reshape(out.shape)))


def _worker(rank, world, port, q_out):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank,
                            world_size=world)
    spec = small_spec(seed=11)
    k, v = wl.pools_np(spec)
    q = wl.q_np(spec)
    t, ln = seqsplit.shard_context(spec.block_tables, spec.seq_lens, rank, world)
    B, H, D = q.shape
    out = torch.zeros((B, H, D), dtype=torch.float64)
    part = torch.zeros(B * H * (D + 2), dtype=torch.float64)
    # bf16 bit patterns travel as uint16 tensors on the CPU
    seqsplit.decode(torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v),
                    torch.from_numpy(t), torch.from_numpy(ln), spec.scale, out, None, part,
                    partial_fn=_oracle_partial_fn, merge_fn=_oracle_merge_fn)
    dist.barrier()
    dist.destroy_process_group()
    q_out.put((rank, out.numpy()))


def test_two_gloo_ranks_reach_the_full_result():
    ctx = mp.get_context("spawn")
    qu = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29633, qu)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((qu.get(timeout=180) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    spec = small_spec(seed=11)
    k, v = wl.pools_np(spec)
    ref = oracle.pa_decode(wl.q_np(spec), k, v, spec.block_tables, spec.seq_lens, spec.scale)
    for _, out in res:  # every rank ends with the whole output
        np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
