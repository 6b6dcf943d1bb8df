"""Sequence-split decode on one GPU: the ranks' slices are attended one after another by
pa_decode_partial (no kernel waits on another), their records merged by pa_merge_partials,
and the result compared with the fp64 oracle of the whole context."""
import numpy as np
import pytest
import torch

import oracle
from oracle import partials
from paper_2602_07878_b200 import api, seqsplit
from paper_2602_07878_b200 import workloads as wl
from helpers import GpuDecode, assert_parity, torch_to_f64

pytestmark = pytest.mark.gpu

LN2 = float(np.log(2.0))


def run_split(spec, world, g=None, partition_tokens=0):
    g = g or GpuDecode(spec)
    B, H, D = g.q.shape
    n = api.pa_partial_floats(api.shape_of(g.k, H), B)
    assert n == (B * H * (D + 2) + 3) // 4 * 4
    gathered = torch.full((world, n), float("nan"), dtype=torch.float32, device="cuda")
    for r in range(world):
        t, ln = seqsplit.shard_context(spec.block_tables, spec.seq_lens, r, world)
        api.pa_decode_partial(g.q, g.k, g.v, torch.from_numpy(t).cuda(),
                              torch.from_numpy(ln).cuda(), spec.scale, gathered[r], g.ws,
                              partition_tokens=partition_tokens, dev_status=g.status)
    g.out.fill_(float("nan"))
    api.pa_merge_partials(gathered, B * H, D, g.out)
    torch.cuda.synchronize()
    assert int(g.status.item()) == 0
    g.check_guards()
    return g, gathered


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("H,Hkv,D", [(8, 2, 128), (4, 4, 64), (16, 8, 256), (16, 1, 128)])
def test_merged_ranks_match_the_oracle(world, H, Hkv, D):
    lens = [1, 15, 16, 17, 33, 0, 70, 129, 513, 1000, 2049, 5000]
    spec = wl.make_spec("t", seq_lens=lens, num_q_heads=H, num_kv_heads=Hkv, head_dim=D,
                        occupancy=0.9, seed=world * 100 + D)
    g, _ = run_split(spec, world)
    k, v = wl.pools_np(spec)
    ref = oracle.pa_decode(wl.q_np(spec), k, v, spec.block_tables, spec.seq_lens, spec.scale)
    out = torch_to_f64(g.out)
    assert_parity(out, ref, f"world {world} H{H}/{Hkv} D{D}")
    assert (out[5] == 0).all()


def test_odd_row_count_keeps_packed_records_aligned():
    spec = wl.make_spec("t", seq_lens=[100, 7, 900], num_q_heads=5, num_kv_heads=5, head_dim=128,
                        occupancy=0.9, seed=3)
    g, gathered = run_split(spec, 3)
    assert gathered.shape[1] == 1952  # 15 rows * 130 floats = 1950, rounded up
    k, v = wl.pools_np(spec)
    ref = oracle.pa_decode(wl.q_np(spec), k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert_parity(torch_to_f64(g.out), ref, "odd rows")


def test_partial_records_match_the_oracle_partials():
    # what is unique in a record: the normalised row o / l and the log-sum-exp m + log l
    lens = [40, 1, 700, 0, 16, 2100]
    spec = wl.make_spec("t", seq_lens=lens, num_q_heads=8, num_kv_heads=2, head_dim=128,
                        occupancy=0.9, seed=77)
    world = 2
    g, gathered = run_split(spec, world)
    B, H, D = g.q.shape
    k, v = wl.pools_np(spec)
    for r in range(world):
        t, ln = seqsplit.shard_context(spec.block_tables, spec.seq_lens, r, world)
        o, m, l = partials.decode_partial(wl.q_np(spec), k, v, t, ln, spec.scale)
        rec = gathered[r].double().cpu().numpy()
        go = rec[: B * H * D].reshape(B, H, D)
        gml = rec[B * H * D:].reshape(B, H, 2)
        empty = ln == 0
        assert np.isneginf(gml[empty, :, 0]).all() and (gml[empty, :, 1] == 0).all()
        assert (go[empty] == 0).all()
        ne = ~empty
        assert_parity(go[ne] / gml[ne, :, 1:2], o[ne] / l[ne][..., None], f"rank {r} rows")
        lse_gpu = gml[ne, :, 0] * LN2 + np.log(gml[ne, :, 1])  # the record keeps m in log2 units
        lse_ref = m[ne] + np.log(l[ne])
        assert np.abs(lse_gpu - lse_ref).max() < 2e-2


def test_one_rank_equals_pa_decode_within_rounding():
    spec = wl.config_spec(1)
    g, _ = run_split(spec, 1)
    split = g.out.clone()
    g.run()
    # same kernels, same partitions; the only difference is one extra fp32 pass for rows that
    # pa_decode writes straight from the attention kernel
    assert_parity(torch_to_f64(split), torch_to_f64(g.out).astype(np.float64), "vs pa_decode",
                  abs_tol=4e-3)


def test_separate_buffers_and_gathered_rows_give_the_same_bits():
    spec = wl.make_spec("t", seq_lens=[300, 45, 1025], num_q_heads=4, num_kv_heads=2,
                        head_dim=128, occupancy=0.9, seed=5)
    g, gathered = run_split(spec, 3)
    ref_bits = g.out.clone().view(torch.int16)
    parts = [gathered[r].clone() for r in (2, 0, 1)]  # separate allocations, another order
    out2 = torch.empty_like(g.out)
    api.pa_merge_partials(parts, g.q.shape[0] * g.q.shape[1], g.q.shape[2], out2)
    torch.cuda.synchronize()
    # the sum over parts is taken in list order, so only the bf16 result is compared
    assert_parity(torch_to_f64(out2), torch_to_f64(g.out), "order of parts", abs_tol=4e-3)
    out3 = torch.empty_like(g.out)
    api.pa_merge_partials([gathered[r].clone() for r in range(3)], 12, 128, out3)
    torch.cuda.synchronize()
    assert torch.equal(out3.view(torch.int16), ref_bits)


def test_bad_block_id_in_one_rank_zeroes_only_that_row():
    spec = wl.make_spec("t", seq_lens=[64, 64, 64], num_q_heads=4, num_kv_heads=4, head_dim=64,
                        occupancy=0.9, seed=8)
    g = GpuDecode(spec)
    B, H, D = g.q.shape
    n = B * H * (D + 2)
    gathered = torch.zeros((2, n), dtype=torch.float32, device="cuda")
    for r in range(2):
        t, ln = seqsplit.shard_context(spec.block_tables, spec.seq_lens, r, 2)
        if r == 1:
            t = t.copy()
            t[1, 0] = spec.num_blocks + 5
        api.pa_decode_partial(g.q, g.k, g.v, torch.from_numpy(t).cuda(),
                              torch.from_numpy(ln).cuda(), spec.scale, gathered[r], g.ws,
                              dev_status=g.status)
    api.pa_merge_partials(gathered, B * H, D, g.out)
    torch.cuda.synchronize()
    assert int(g.status.item()) & api.PA_STATUS_BAD_BLOCK_ID
    out = torch_to_f64(g.out)
    k, v = wl.pools_np(spec)
    ref = oracle.pa_decode(wl.q_np(spec), k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert (out[1] == 0).all()
    assert_parity(out[[0, 2]], ref[[0, 2]], "other rows")


def test_merge_argument_errors():
    out = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    part = torch.zeros(4 * 66, dtype=torch.float32, device="cuda")
    with pytest.raises(api.PagedKVError):
        api.pa_merge_partials([part] * 33, 4, 64, out)  # more than PA_MAX_PARTS
    assert api.lib().pa_merge_partials(None, 1, 4, 96, out.data_ptr(), None) == api.ERR["SHAPE"]
    # no parts: every row is zeros
    out.fill_(1.0)
    api.pa_merge_partials([], 4, 64, out)
    torch.cuda.synchronize()
    assert (out == 0).all()
