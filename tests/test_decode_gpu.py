"""GPU parity of pa_decode (through the C-ABI) against the fp64 CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from helpers import GpuDecode, assert_parity, oracle_for, torch_to_f64, bits_to_torch

pytestmark = pytest.mark.gpu


def small_inputs(spec, poison=True):
    q = wl.q_np(spec)
    k, v = wl.pools_np(spec, poison_tails=poison)
    return q, k, v


def run_and_check(spec, partition_tokens=0, what=""):
    q, k, v = small_inputs(spec)
    g = GpuDecode(spec, q, k, v, partition_tokens=partition_tokens)
    out = torch_to_f64(g.run())
    ref = oracle_for(spec, q, k, v)
    assert int(g.status.item()) == 0
    return assert_parity(out, ref, what or spec.name), g, out, ref


def test_cfg1_tiny_mha_matches_oracle():
    rel, g, out, ref = run_and_check(wl.config_spec(1))
    assert rel < 1e-2        # bf16 output rounding is ~2^-9 of the row maximum
    # the same comparison against the stored oracle values (tests/golden)
    from test_golden_cpu import load_golden
    for b, h, d, x in load_golden():
        assert abs(out[b, h, d] - x) <= 1e-2


@pytest.mark.parametrize("P", [16, 32, 64, 128, 512])
def test_cfg1_forced_partitions(P):
    run_and_check(wl.config_spec(1), partition_tokens=P)


@pytest.mark.parametrize("H,Hkv,D", [(4, 4, 64), (8, 2, 64), (8, 2, 128), (32, 8, 128),
                                     (8, 1, 128), (16, 1, 128), (32, 2, 64), (6, 3, 128),
                                     (12, 1, 64), (5, 5, 128), (16, 8, 256), (4, 4, 256),
                                     (16, 1, 256), (6, 2, 256)])
def test_head_layouts(H, Hkv, D):
    lens = [1, 15, 16, 17, 31, 33, 0, 70, 129, 513, 1000, 2049]
    spec = wl.make_spec("t", seq_lens=lens, num_q_heads=H, num_kv_heads=Hkv, head_dim=D,
                        occupancy=0.9, seed=H * 1000 + Hkv * 10 + D)
    for P in (0, 64, 512):
        _, g, out, ref = run_and_check(spec, partition_tokens=P, what=f"H{H}/{Hkv} D{D} P{P}")
        assert (out[6] == 0).all()


def test_more_sequences_than_the_plan_kernel_has_threads():
    # 2300 sequences: the plan walks them in three rounds of its 1024 threads, and only the
    # first round's sequences have their lengths in the plan's shared memory; long sequences
    # sit in every round so that split and unsplit rows come from both paths
    rng = np.random.default_rng(5)
    lens = rng.integers(0, 60, size=2300)
    lens[[3, 1023, 1024, 1500, 2299]] = [700, 1300, 900, 2048, 513]
    spec = wl.make_spec("t", seq_lens=lens, num_q_heads=4, num_kv_heads=2, head_dim=64,
                        occupancy=0.95, seed=23)
    for P in (0, 128):
        run_and_check(spec, partition_tokens=P, what=f"2300 sequences P{P}")


def test_many_short_and_ragged_sequences_span_all_warps():
    rng = np.random.default_rng(1)
    lens = rng.integers(0, 200, size=700)
    spec = wl.make_spec("t", seq_lens=lens, num_q_heads=8, num_kv_heads=4, head_dim=128,
                        occupancy=0.97, seed=21)
    run_and_check(spec)


def test_mixed_long_and_short_scaled_cfg3():
    spec = wl.config_spec(3, scale_down=8)       # 1 x 32768 + 31 lognormal, GQA 32/8
    rel, g, out, ref = run_and_check(spec)
    hdr = g.plan_header()
    assert hdr[0] > spec.batch                   # the long sequence was split
    for P in (256, 512):
        run_and_check(spec, partition_tokens=P)


def test_output_is_bit_identical_under_block_permutation_and_batch_order():
    spec = wl.config_spec(1)
    q, k, v = small_inputs(spec)
    base = GpuDecode(spec, q, k, v, partition_tokens=64).run().clone()
    rng = np.random.default_rng(5)
    perm = rng.permutation(spec.num_blocks)
    k2, v2 = np.empty_like(k), np.empty_like(v)
    k2[perm], v2[perm] = k, v
    t2 = spec.block_tables.copy()
    for b in range(spec.batch):
        nb = len(spec.blocks_of(b))
        t2[b, :nb] = perm[spec.block_tables[b, :nb]]
    out2 = GpuDecode(spec, q, k2, v2, tables=t2, partition_tokens=64).run()
    assert torch.equal(out2.view(torch.int16), base.view(torch.int16))
    order = [3, 1, 0, 2]
    out3 = GpuDecode(spec, q[order], k, v, tables=spec.block_tables[order],
                     lens=spec.seq_lens[order], partition_tokens=64).run()
    assert torch.equal(out3.view(torch.int16), base[order].view(torch.int16))
    # repeated runs reproduce bit for bit
    g = GpuDecode(spec, q, k, v)
    a = g.run().clone()
    assert torch.equal(g.run().view(torch.int16), a.view(torch.int16))


def test_single_token_returns_value_bits():
    spec = wl.make_spec("t", seq_lens=[1, 1, 1], num_q_heads=8, num_kv_heads=4, head_dim=128,
                        num_blocks=6, seed=31)
    q, k, v = small_inputs(spec)
    out = GpuDecode(spec, q, k, v).run().view(torch.int16).cpu().numpy().view(np.uint16)
    for b in range(3):
        p = int(spec.block_tables[b, 0])
        for h in range(8):
            assert (out[b, h] == v[p, h // 2, 0]).all()


def test_equal_keys_give_mean_of_values():
    spec = wl.make_spec("t", seq_lens=[37, 640], num_q_heads=4, num_kv_heads=2, head_dim=64,
                        occupancy=0.9, seed=32)
    q, k, v = small_inputs(spec)
    k[:] = wl.normal_bf16_np(0, 64, 999)
    g = GpuDecode(spec, q, k, v, partition_tokens=128)
    out = torch_to_f64(g.run())
    ref = oracle_for(spec, q, k, v)
    assert_parity(out, ref)


def test_large_scores_do_not_overflow():
    spec = wl.make_spec("t", seq_lens=[300, 45], num_q_heads=4, num_kv_heads=4, head_dim=128,
                        occupancy=0.9, seed=33)
    q, k, v = small_inputs(spec)
    for scale in (8.0, -8.0):                 # |scores| up to a few hundred
        g = GpuDecode(spec, q, k, v, partition_tokens=64)
        out = torch_to_f64(g.run(scale=scale))
        ref = oracle_for(spec, q, k, v, scale=scale)
        assert_parity(out, ref, f"scale {scale}")


def test_shared_prefix_block():
    spec = wl.make_spec("t", seq_lens=[40, 40], num_q_heads=2, num_kv_heads=2, head_dim=64,
                        num_blocks=8, seed=12)
    q, k, v = small_inputs(spec)
    t = spec.block_tables.copy()
    t[1, 0] = t[0, 0]
    out = torch_to_f64(GpuDecode(spec, q, k, v, tables=t).run())
    assert_parity(out, oracle_for(spec, q, k, v, tables=t))


def test_strided_cache_layout():
    # cache stored [NB, bs, Hkv, D] (token-major) and passed as a strided [NB, Hkv, bs, D] view
    spec = wl.make_spec("t", seq_lens=[100, 700, 16], num_q_heads=8, num_kv_heads=2,
                        head_dim=128, occupancy=0.9, seed=34)
    q, k, v = small_inputs(spec)
    g = GpuDecode(spec, q, k, v)
    g.k = g.k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    g.v = g.v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not g.k.is_contiguous()
    out = torch_to_f64(g.run())
    assert_parity(out, oracle_for(spec, q, k, v))


def test_bad_lengths_and_block_ids_are_reported_and_rows_zeroed():
    spec = wl.config_spec(1)
    q, k, v = small_inputs(spec)
    ref = oracle_for(spec, q, k, v)
    lens = spec.seq_lens.copy()
    lens[1] = spec.max_blocks * 16 + 1
    g = GpuDecode(spec, q, k, v, lens=lens)
    out = torch_to_f64(g.run())
    assert int(g.status.item()) == api.PA_STATUS_BAD_SEQ_LEN
    assert (out[1] == 0).all()
    assert_parity(out[[0, 2, 3]], ref[[0, 2, 3]])
    for P in (0, 64):
        t = spec.block_tables.copy()
        t[3, 5] = spec.num_blocks        # one past the pool
        t[0, 1] = -7
        g = GpuDecode(spec, q, k, v, tables=t, partition_tokens=P)
        out = torch_to_f64(g.run())
        assert int(g.status.item()) == api.PA_STATUS_BAD_BLOCK_ID
        assert (out[3] == 0).all() and (out[0] == 0).all()
        assert_parity(out[[1, 2]], ref[[1, 2]])


def test_reuse_plan_flag_and_other_stream():
    spec = wl.config_spec(3, scale_down=8)
    q, k, v = small_inputs(spec)
    g = GpuDecode(spec, q, k, v)
    a = g.run().clone()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for _ in range(3):
            b = g.run(flags=api.PA_FLAG_REUSE_PLAN, stream=s).clone()
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_back_to_back_calls_with_different_plans_share_a_workspace():
    """The plan kernel of a call runs beside the combine kernel of the call before it and fills
    the plan region that call does not use.  Calls with different length sets (so different
    work lists, partition counts and combine lists) are queued on one stream and one workspace
    with no synchronisation in between; every call's rows must be the ones it gives alone."""
    spec = wl.config_spec(3, scale_down=8)
    q, k, v = small_inputs(spec)
    g = GpuDecode(spec, q, k, v)
    rng = np.random.default_rng(11)
    base = spec.seq_lens.astype(np.int64)
    variants = []
    for i in range(5):
        lens = base.copy()
        pick = rng.random(lens.size)
        lens[pick < 0.3] = 0                                  # rows of zeros through the combine
        lens[(pick >= 0.3) & (pick < 0.6)] //= int(rng.integers(2, 9))
        if i == 3:
            lens[:] = np.minimum(lens, 40)                    # every sequence a single partition
        variants.append(lens.astype(np.int32))
    alone = []
    for lens in variants:
        g.lens.copy_(torch.from_numpy(lens).cuda())
        alone.append(g.run().clone())
        assert int(g.status.item()) == 0
    ref = oracle.pa_decode(q, k, v, spec.block_tables, variants[1], spec.scale)
    assert_parity(torch_to_f64(alone[1]), ref, "variant 1 alone")

    dev_lens = [torch.from_numpy(l).cuda() for l in variants]
    outs = [torch.full_like(g.q, float("nan")) for _ in range(12)]
    order = [0, 1, 2, 3, 4, 3, 1, 1, 0, 4, 2, 0]
    torch.cuda.synchronize()
    for out, which in zip(outs, order):
        api.pa_decode(g.q, g.k, g.v, g.tables, dev_lens[which], spec.scale, out, g.ws,
                      dev_status=g.status)
    # a call that keeps the plan of the call before it, then one that plans again
    again = torch.full_like(g.q, float("nan"))
    api.pa_decode(g.q, g.k, g.v, g.tables, dev_lens[order[-1]], spec.scale, again, g.ws,
                  dev_status=g.status, flags=api.PA_FLAG_REUSE_PLAN)
    last = torch.full_like(g.q, float("nan"))
    api.pa_decode(g.q, g.k, g.v, g.tables, dev_lens[2], spec.scale, last, g.ws, dev_status=g.status)
    torch.cuda.synchronize()
    assert int(g.status.item()) == 0
    g.check_guards()
    for out, which in zip(outs + [again, last], order + [order[-1], 2]):
        assert torch.equal(out.view(torch.int16), alone[which].view(torch.int16)), which


def test_workspace_too_small_for_plan_is_reported():
    spec = wl.make_spec("t", seq_lens=[4096] * 8, num_q_heads=8, num_kv_heads=8, head_dim=64,
                        occupancy=0.9, seed=35)
    q, k, v = small_inputs(spec)
    g = GpuDecode(spec, q, k, v, max_tokens=4096, partition_tokens=16)  # cap far below need
    out = torch_to_f64(g.run())
    assert int(g.status.item()) & api.PA_STATUS_WORKSPACE
    assert (out == 0).all()


def test_pa_decode_host_matches_device_call():
    spec = wl.config_spec(1)
    q, k, v = small_inputs(spec)
    g = GpuDecode(spec, q, k, v)
    dev_out = g.run().cpu()
    qh = g.q.cpu().pin_memory()
    th = g.tables.cpu().pin_memory()
    lh = g.lens.cpu().pin_memory()
    oh = torch.zeros_like(qh).pin_memory()
    shape = api.shape_of(g.k, 8)
    io = torch.empty(api.pa_host_io_bytes(shape, 4, th.shape[1]), dtype=torch.uint8, device="cuda")
    api.pa_decode_host(qh, g.k, g.v, th, lh, spec.scale, oh, io, g.ws)
    torch.cuda.synchronize()
    assert torch.equal(oh.view(torch.int16), dev_out.view(torch.int16))


def test_pa_decode_host_reads_large_tables_in_place():
    # [32, 2048] int32 tables are 256 KiB: read in place over the host link, output posted in place
    spec = wl.config_spec(3, scale_down=8)
    q, k, v = small_inputs(spec)
    g = GpuDecode(spec, q, k, v)
    dev_out = g.run().cpu()
    qh, th, lh = g.q.cpu().pin_memory(), g.tables.cpu().pin_memory(), g.lens.cpu().pin_memory()
    assert th.numel() * 4 >= 256 << 10
    oh = torch.zeros_like(qh).pin_memory()
    shape = api.shape_of(g.k, spec.num_q_heads)
    io = torch.empty(api.pa_host_io_bytes(shape, spec.batch, th.shape[1]), dtype=torch.uint8,
                     device="cuda")
    for _ in range(2):
        api.pa_decode_host(qh, g.k, g.v, th, lh, spec.scale, oh, io, g.ws, dev_status=g.status)
        torch.cuda.synchronize()
        assert torch.equal(oh.view(torch.int16), dev_out.view(torch.int16))
    assert int(g.status.item()) == 0


@pytest.mark.parametrize("D,pinned", [(128, False), (256, True), (64, True)])
def test_pa_decode_host_copies_what_it_cannot_read_in_place(D, pinned):
    # pageable host tensors go through the device staging buffer (q always does); pinned
    # tables and outputs of other head dims take the same call
    spec = wl.make_spec("t", seq_lens=[40, 700, 0, 1300, 17], num_q_heads=8, num_kv_heads=2,
                        head_dim=D, occupancy=0.9, seed=31 + D)
    q, k, v = small_inputs(spec)
    g = GpuDecode(spec, q, k, v)
    dev_out = g.run().cpu()
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    qh, th, lh = pin(g.q.cpu()), pin(g.tables.cpu()), pin(g.lens.cpu())
    oh = pin(torch.zeros_like(g.q.cpu()))
    shape = api.shape_of(g.k, spec.num_q_heads)
    io = torch.empty(api.pa_host_io_bytes(shape, spec.batch, th.shape[1]), dtype=torch.uint8,
                     device="cuda")
    api.pa_decode_host(qh, g.k, g.v, th, lh, spec.scale, oh, io, g.ws, dev_status=g.status)
    torch.cuda.synchronize()
    assert torch.equal(oh.view(torch.int16), dev_out.view(torch.int16))
    assert int(g.status.item()) == 0


def test_a_wait_that_nobody_completes_times_out_and_reports_it():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    api.pa_selftest_wait_expiry(2000, status)            # 2 ms limit
    e1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == api.PA_STATUS_TIMEOUT
    assert 1.5 < e0.elapsed_time(e1) < 100.0             # gave up after the limit, not much later
    # the context is still usable
    spec = wl.config_spec(1)
    q, k, v = small_inputs(spec)
    assert_parity(torch_to_f64(GpuDecode(spec, q, k, v).run()), oracle_for(spec, q, k, v))


def test_read_probes_run_and_report_no_timeout():
    buf = torch.zeros(64 << 20, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    n0 = api.pa_launch_count()
    api.pa_probe_read(buf, False, status)
    api.pa_probe_read(buf, True, status, seed=7)
    api.pa_probe_read(buf[: 4096 * 3], True, status)      # fewer granules than warps
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and api.pa_launch_count() - n0 == 3


@pytest.mark.parametrize("warps,boxes", [(1, 16), (4, 4), (8, 2), (2, 2)])
def test_tma_issue_probe_runs_and_counts_its_boxes(warps, boxes):
    buf = torch.zeros(8 << 20, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    n = api.pa_probe_tma_issue(buf, warps, boxes, 3, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # every warp of every SM issues the same number of slots; the whole buffer is covered 3 times
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert n % (sms * warps * boxes) == 0 and n * 2048 >= 3 * buf.numel()


def test_a_batch_of_empty_sequences_gives_zero_rows():
    # nothing allocated at all: the pool still has a block, every output row is zeros
    spec = wl.make_spec("t", seq_lens=[0, 0, 0], num_q_heads=8, num_kv_heads=8, head_dim=64,
                        occupancy=1.0, seed=3)
    assert spec.num_blocks == 1
    _, g, out, ref = run_and_check(spec)
    assert (out == 0).all() and int(g.status.item()) == 0
