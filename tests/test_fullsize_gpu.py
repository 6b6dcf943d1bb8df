"""Parity at the full workload sizes, in the launch configuration bench.py times
(automatic partition size, device-generated inputs): sampled sequences are recomputed by the
fp64 oracle from inputs regenerated on the CPU; properties that hold for every row are
checked on all rows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from helpers import abs_bits, assert_parity, torch_to_f64

pytestmark = pytest.mark.gpu


def host_inputs_for(spec, seqs, layer=0):
    """q rows, compact K/V pools and remapped tables of `seqs`, regenerated with numpy."""
    ids = np.concatenate([spec.blocks_of(b) for b in seqs]).astype(np.int64)
    remap = {int(p): i for i, p in enumerate(ids)}
    k = wl.pool_block_np(spec, "k", ids, layer)
    v = wl.pool_block_np(spec, "v", ids, layer)
    if layer == 0:
        for blk, slot in wl.tail_slots(spec):
            if blk in remap:
                k[remap[blk], :, slot:] = wl.BF16_NAN_BITS
                v[remap[blk], :, slot:] = wl.BF16_NAN_BITS
    mb = max(len(spec.blocks_of(b)) for b in seqs)
    tables = np.zeros((len(seqs), mb), np.int32)
    for i, b in enumerate(seqs):
        blk = spec.blocks_of(b)
        tables[i, :len(blk)] = [remap[int(p)] for p in blk]
    H, D = spec.num_q_heads, spec.head_dim
    q = np.stack([wl.normal_bf16_np(b * H * D, H * D, spec.seed_q).reshape(H, D) for b in seqs])
    return q, k, v, tables, spec.seq_lens[seqs].astype(np.int32), ids


def pick(spec, n_long, n_other, seed=3):
    rng = np.random.default_rng(seed)
    order = np.argsort(-spec.seq_lens.astype(np.int64), kind="stable")
    longs = [int(b) for b in order[:n_long]]
    rest = [int(b) for b in rng.permutation(order[n_long:])[:n_other]]
    shortest = int(order[-1])
    return sorted(set(longs + rest + [shortest]))


def decode_full(spec, k, v, q=None):
    dev = "cuda"
    q = wl.q_torch(spec, dev) if q is None else q
    tables = torch.from_numpy(spec.block_tables).to(dev)
    lens = torch.from_numpy(spec.seq_lens).to(dev)
    out = torch.full_like(q, float("nan"))
    shape = api.shape_of(k, spec.num_q_heads)
    ws = torch.empty(api.pa_workspace_bytes(shape, spec.batch, spec.total_tokens + 16 * spec.batch),
                     dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    api.pa_decode(q, k, v, tables, lens, spec.scale, out, ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    hdr = ws[:256].view(torch.int32).cpu().numpy()
    return q, out, hdr


@pytest.mark.parametrize("index,n_long,n_other", [(2, 2, 6), (3, 1, 12), (5, 1, 2)])
def test_full_size_decode_sampled_against_oracle(index, n_long, n_other):
    spec = wl.config_spec(index)
    k, v = wl.pools_torch(spec, "cuda")
    q, out, hdr = decode_full(spec, k, v)
    # every row: finite, and a convex mixture of N(0,1)-table values cannot leave their range
    assert torch.isfinite(out).all()
    assert float(out.float().abs().max()) <= 4.25
    assert int(hdr[0]) >= spec.batch and int(hdr[2]) in (64, 128, 256, 512)
    seqs = pick(spec, n_long, n_other)
    qh, kh, vh, tables, lens, ids = host_inputs_for(spec, seqs)
    # the device generator and the host generator give the same bits
    some = ids[:: max(1, len(ids) // 16)]
    dev_bits = k[torch.from_numpy(some).cuda()].view(torch.int16).cpu().numpy().view(np.uint16)
    assert (dev_bits == kh[:: max(1, len(ids) // 16)]).all()
    assert (q[seqs].view(torch.int16).cpu().numpy().view(np.uint16) == qh).all()
    ref = oracle.pa_decode(qh, kh, vh, tables, lens, spec.scale)
    assert_parity(torch_to_f64(out[seqs]), ref, spec.name)


@pytest.mark.parametrize("index", [2, 3, 5])
def test_full_size_host_call_gives_the_device_call_bits(index):
    # pa_decode_host at the bench's sizes: workloads 2 and 3 read q in place from pinned host
    # memory (the host-memory instantiation of the attention kernel), workload 5 copies it
    spec = wl.config_spec(index)
    k, v = wl.pools_torch(spec, "cuda")
    q, out, hdr = decode_full(spec, k, v)
    tables = torch.from_numpy(spec.block_tables).pin_memory()
    lens = torch.from_numpy(spec.seq_lens).pin_memory()
    qh = q.cpu().pin_memory()
    oh = torch.zeros_like(qh).pin_memory()
    shape = api.shape_of(k, spec.num_q_heads)
    io = torch.empty(api.pa_host_io_bytes(shape, spec.batch, tables.shape[1]), dtype=torch.uint8,
                     device="cuda")
    ws = torch.empty(api.pa_workspace_bytes(shape, spec.batch, spec.total_tokens + 16 * spec.batch),
                     dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(2):
        oh.zero_()
        api.pa_decode_host(qh, k, v, tables, lens, spec.scale, oh, io, ws, dev_status=status)
        torch.cuda.synchronize()
        assert torch.equal(oh.view(torch.int16), out.cpu().view(torch.int16))
    assert int(status.item()) == 0


def test_full_size_swap_churn_and_decode():
    """Workload 4 at full size: 32-layer pool of 60000 blocks at 98 % occupancy; evict 64K
    tokens' worth of whole sequences, restore them into other blocks, decode one layer."""
    free, total = torch.cuda.mem_get_info()
    if free < 150 * (1 << 30):
        pytest.skip("needs about 140 GB of free device memory")
    spec = wl.config_spec(4)
    dev = "cuda"
    layers, nb = spec.num_layers, spec.num_blocks
    n = nb * spec.block_elems
    shape5 = (layers, nb, spec.num_kv_heads, 16, spec.head_dim)
    k_pool = wl.normal_bf16_torch(0, layers * n, spec.seed_k, dev).view(shape5)
    v_pool = wl.normal_bf16_torch(0, layers * n, spec.seed_v, dev).view(shape5)
    seqs, src, dst = wl.pick_victims(spec, 65536, seed=11)
    assert len(src) == 4096 and len(set(dst.tolist())) == 4096
    bb = api.kv_block_bytes(k_pool, v_pool)
    assert bb == 2 << 20
    host = torch.empty(len(src) * bb, dtype=torch.uint8, pin_memory=True)
    staging = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def checksum(exclude):
        keep = torch.ones(nb, dtype=torch.bool, device=dev)
        keep[torch.from_numpy(np.asarray(exclude, dtype=np.int64)).to(dev)] = False
        tot = 0
        for pool in (k_pool, v_pool):
            for l in range(layers):
                x = pool[l].view(torch.int16).view(nb, -1)
                tot += int((x.sum(dim=1, dtype=torch.int64) * keep).sum().item())
        return tot

    before = checksum(dst)
    api.kv_swap_out(k_pool, v_pool, src, host, staging)
    torch.cuda.synchronize()
    img = host.numpy().view(np.uint16).reshape(len(src), layers, 2, -1)
    rng = np.random.default_rng(0)
    for i in rng.integers(0, len(src), 6):
        for layer in (0, 13, 31):
            assert (img[i, layer, 0] == wl.pool_block_np(spec, "k", [src[i]], layer).reshape(-1)).all()
            assert (img[i, layer, 1] == wl.pool_block_np(spec, "v", [src[i]], layer).reshape(-1)).all()
    src_t = torch.from_numpy(src.astype(np.int64)).to(dev)
    dst_t = torch.from_numpy(dst.astype(np.int64)).to(dev)
    # the freed blocks get overwritten before the victims come back (unless reused as targets)
    reused = set(dst.tolist())
    trash = torch.from_numpy(np.array([p for p in src if p not in reused], dtype=np.int64)).to(dev)
    expect_k = k_pool[:, src_t].clone()
    expect_v = v_pool[:, src_t].clone()
    trash_sum = sum(int(p[:, trash].view(torch.int16).sum(dtype=torch.int64).item())
                    for p in (k_pool, v_pool))
    k_pool[:, trash] = float("nan")
    v_pool[:, trash] = float("nan")
    api.kv_swap_in(k_pool, v_pool, host, dst, None)          # direct mode on the way back
    torch.cuda.synchronize()
    assert torch.equal(k_pool[:, dst_t].view(torch.int16), expect_k.view(torch.int16))
    assert torch.equal(v_pool[:, dst_t].view(torch.int16), expect_v.view(torch.int16))
    del expect_k, expect_v
    # bytes outside the destination blocks did not change (the trashed ones are zeroed and
    # their original content, summed on the device beforehand, is subtracted)
    k_pool[:, trash] = 0
    v_pool[:, trash] = 0
    after = checksum(dst)
    before_adj = before - trash_sum
    assert after == before_adj

    # decode layer 7 over the whole batch with the victims remapped to their new blocks
    layer = 7
    t = spec.block_tables.copy()
    o = 0
    for b in seqs:
        nblk = min(len(spec.blocks_of(b)), len(dst) - o)
        t[b, :nblk] = dst[o:o + nblk]
        o += nblk
    spec2 = wl.DecodeSpec(**{**spec.__dict__, "block_tables": t})
    q, out, hdr = decode_full(spec2, k_pool[layer], v_pool[layer])
    assert torch.isfinite(out).all()
    sample = sorted(set(pick(spec, 1, 4) + seqs[:2]))
    # oracle inputs from the CPU generator at the ORIGINAL block ids (content moved with the swap)
    qh, kh, vh, tables, lens, ids = host_inputs_for(spec, sample, layer)
    ref = oracle.pa_decode(qh, kh, vh, tables, lens, spec.scale)
    assert_parity(torch_to_f64(out[sample]), ref, "workload 4 decode after churn")


def test_decode_time_is_linear_in_total_context_once_bandwidth_bound():
    """Eq. 3 of the paper models the attention step's time as context bytes / HBM bandwidth.
    Doubling every context length must therefore about double the step's device time once
    the batch is far larger than L2."""
    times = {}
    for mult in (1, 2, 4):
        lens = np.full(96, 2048 * mult, np.int64)
        spec = wl.make_spec("t", seq_lens=lens, num_q_heads=32, num_kv_heads=8, head_dim=128,
                            occupancy=0.97, seed=mult)
        n = spec.num_blocks * spec.block_elems
        shape = (spec.num_blocks, 8, 16, 128)
        k = wl.normal_bf16_torch(0, n, 1, "cuda").view(shape)
        v = wl.normal_bf16_torch(0, n, 2, "cuda").view(shape)
        q = wl.q_torch(spec, "cuda")
        tables = torch.from_numpy(spec.block_tables).cuda()
        lens_d = torch.from_numpy(spec.seq_lens).cuda()
        out = torch.empty_like(q)
        ws = torch.empty(api.pa_workspace_bytes(api.shape_of(k, 32), 96, spec.total_tokens + 2048),
                         dtype=torch.uint8, device="cuda")
        for _ in range(3):
            api.pa_decode(q, k, v, tables, lens_d, spec.scale, out, ws)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            api.pa_decode(q, k, v, tables, lens_d, spec.scale, out, ws)
        e1.record()
        e1.synchronize()
        times[mult] = e0.elapsed_time(e1) / 20
        assert spec.kv_bytes() > 4 * (126 << 20)
        del k, v
    assert 1.8 < times[2] / times[1] < 2.2, times
    assert 1.8 < times[4] / times[2] < 2.2, times


@pytest.mark.parametrize("H,Hkv,D,chunk", [(32, 8, 128, 512), (32, 8, 128, 32768), (16, 8, 256, 512),
                                           (16, 8, 256, 8192)])
def test_full_size_recompute_sampled_against_oracle(H, Hkv, D, chunk):
    """The recompute leg of bench.py at its sizes: the last `chunk` query tokens of a
    32768-token context over a shuffled block table, launched as the bench launches it
    (library-chosen tile count and KV split, workspace for 16 splits).  The oracle recomputes
    sampled query tokens one by one -- a query at position p is a decode step over p + 1 tokens
    -- on the first and last rows of the chunk, around tile and split boundaries and at random."""
    L, dev = 32768, "cuda"
    nb = L // 16
    kb = wl.normal_bf16_np(0, (nb + 64) * Hkv * 16 * D, 901).reshape(nb + 64, Hkv, 16, D)
    vb = wl.normal_bf16_np(0, (nb + 64) * Hkv * 16 * D, 902).reshape(nb + 64, Hkv, 16, D)
    table = np.random.default_rng(903).permutation(nb + 64)[:nb].astype(np.int32).reshape(1, nb)
    qb = wl.normal_bf16_np(0, chunk * H * D, 904).reshape(chunk, H, D)
    from helpers import bits_to_torch
    k, v, q = bits_to_torch(kb), bits_to_torch(vb), bits_to_torch(qb)
    out = torch.full_like(q, float("nan"))
    ws = torch.empty(api.pa_prefill_split_workspace_bytes(api.shape_of(k, H), 1, chunk, 16),
                     dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    api.pa_prefill_split(q, k, v, torch.from_numpy(table).to(dev),
                         torch.tensor([L], dtype=torch.int32, device=dev),
                         torch.tensor([0, chunk], dtype=torch.int32, device=dev), D ** -0.5, out, ws,
                         dev_status=status)
    torch.cuda.synchronize()
    tiles, split_tok, splits = api.pa_prefill_last_launch()
    assert int(status.item()) == 0 and tiles in (1, 2)
    if chunk == 512:
        assert splits >= 2                       # few tiles, long context: the KV range is split
    assert torch.isfinite(out).all()
    # rows are convex mixtures of table values
    assert float(out.float().abs().max()) <= float(v.float().abs().max())
    rng = np.random.default_rng(905)
    tpt = 128 // (H // Hkv)
    picks = {0, 1, chunk - 1, chunk - 2, tpt - 1, tpt, 2 * tpt - 1, 2 * tpt, chunk // 2}
    if split_tok:                                # queries whose position sits at a split boundary
        first = L - chunk
        for s in range(1, splits):
            t = s * split_tok - first
            picks |= {x for x in (t - 1, t, t + 1) if 0 <= x < chunk}
    picks |= {int(x) for x in rng.integers(0, chunk, 8)}
    toks = sorted(picks)
    pos = np.array([L - chunk + t for t in toks], np.int32)
    ref = oracle.pa_decode(qb[toks], kb, vb, np.repeat(table, len(toks), axis=0), pos + 1,
                           np.float32(D ** -0.5))
    assert_parity(torch_to_f64(out[toks]), ref, f"recompute H{H}/{Hkv} D{D} chunk {chunk}",
                  amended=lambda: oracle.pa_decode(qb[toks], kb, abs_bits(vb),
                                                   np.repeat(table, len(toks), axis=0), pos + 1,
                                                   np.float32(D ** -0.5)))
