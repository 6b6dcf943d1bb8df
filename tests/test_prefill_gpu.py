"""GPU parity of pa_prefill (through the C-ABI) against the fp64 prefill oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from helpers import abs_bits, assert_parity, bits_to_torch, prefill_ref, torch_to_f64

pytestmark = pytest.mark.gpu


class GpuPrefill:
    def __init__(self, spec, q_bits, k_bits, v_bits, max_splits=0):
        self.spec = spec
        self.q = bits_to_torch(q_bits)
        self.k, self.v = bits_to_torch(k_bits), bits_to_torch(v_bits)
        self.tables = torch.from_numpy(spec.block_tables).cuda()
        nbytes = api.pa_prefill_workspace_bytes(spec.batch)
        if max_splits:
            nbytes = api.pa_prefill_split_workspace_bytes(
                api.shape_of(self.k, q_bits.shape[1]), spec.batch, q_bits.shape[0], max_splits)
        # NaN-filled: a partial record that is read without having been written shows up
        self.ws = torch.full((nbytes // 4,), float("nan"), dtype=torch.float32, device="cuda")
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def run(self, ctx, cu, q=None, tables=None, split=None):
        q = self.q if q is None else q
        out = torch.full_like(q, float("nan"))
        args = (q, self.k, self.v, self.tables if tables is None else tables,
                torch.from_numpy(np.asarray(ctx, np.int32)).cuda(),
                torch.from_numpy(np.asarray(cu, np.int32)).cuda(), self.spec.scale, out, self.ws)
        if split is None:
            api.pa_prefill(*args, dev_status=self.status)
        else:
            api.pa_prefill_split(*args, kv_split_tokens=split, dev_status=self.status)
        torch.cuda.synchronize()
        return out


def make_case(ctx, qlens, H, Hkv, D, seed):
    spec = wl.make_spec("t", seq_lens=ctx, num_q_heads=H, num_kv_heads=Hkv, head_dim=D,
                        occupancy=0.85, seed=seed)
    k, v = wl.pools_np(spec)
    cu = np.concatenate([[0], np.cumsum(qlens)]).astype(np.int32)
    q = wl.normal_bf16_np(0, int(cu[-1]) * H * D, 700 + seed).reshape(int(cu[-1]), H, D)
    return spec, q, k, v, cu


@pytest.mark.parametrize("H,Hkv,D", [(8, 8, 64), (8, 2, 128), (32, 8, 128), (16, 1, 128),
                                     (6, 2, 64), (10, 2, 128), (8, 1, 64), (4, 4, 128),
                                     (8, 4, 128), (8, 1, 128), (64, 8, 128), (16, 8, 256),
                                     (4, 1, 256)])
def test_mixed_chunks_match_oracle(H, Hkv, D):
    ctx = [37, 64, 5, 130, 1, 700, 16, 333]
    qlens = [37, 10, 0, 33, 1, 512, 16, 1]
    spec, q, k, v, cu = make_case(ctx, qlens, H, Hkv, D, seed=H + Hkv + D)
    g = GpuPrefill(spec, q, k, v)
    out = torch_to_f64(g.run(spec.seq_lens, cu))
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert int(g.status.item()) == 0
    assert api.pa_prefill_last_launch()[0] in (1, 2)   # every supported shape runs on tcgen05
    assert_parity(out, ref, f"H{H}/{Hkv} D{D}", amended=abs_ref)


def test_warp_mma_kernel_in_a_child_process():
    # PAGEDKV_PREFILL=mma (read once per process) selects the warp-level MMA kernel
    import os, subprocess, sys, textwrap
    code = textwrap.dedent("""
        import sys
        sys.path.insert(0, "tests")
        import numpy as np, torch
        import oracle
        from paper_2602_07878_b200 import api
        from test_prefill_gpu import GpuPrefill, make_case
        from helpers import assert_parity, prefill_ref, torch_to_f64
        for H, Hkv, D in [(8, 2, 128), (6, 2, 64), (16, 8, 256)]:
            spec, q, k, v, cu = make_case([37, 64, 5, 130, 1, 700], [37, 10, 0, 33, 1, 300], H, Hkv, D, seed=3)
            g = GpuPrefill(spec, q, k, v)
            out = torch_to_f64(g.run(spec.seq_lens, cu))
            assert api.pa_prefill_last_launch()[0] == 0
            ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
            assert int(g.status.item()) == 0
            assert_parity(out, ref, f"warp MMA H{H}/{Hkv} D{D}", amended=abs_ref)
        print("child ok")
    """)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", code], cwd=root, capture_output=True, text=True,
                         env=dict(os.environ, PAGEDKV_PREFILL="mma"), timeout=600)
    assert res.returncode == 0 and "child ok" in res.stdout, res.stdout + res.stderr


def test_single_query_token_equals_decode_bits():
    # a chunk of one query token per sequence is a decode step
    spec, q, k, v, cu = make_case([90, 17, 256], [1, 1, 1], 8, 2, 128, seed=9)
    g = GpuPrefill(spec, q, k, v)
    out = torch_to_f64(g.run(spec.seq_lens, cu))
    ref = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert_parity(out, ref, amended=lambda: oracle.pa_decode(q, k, abs_bits(v), spec.block_tables,
                                                             spec.seq_lens, spec.scale))


def test_chunked_recompute_of_a_long_sequence():
    """Recompute a 3000-token victim in 512-token chunks; every chunk sees the cache up to its
    own end.  The concatenation equals the one-shot oracle."""
    spec, q, k, v, cu = make_case([3000], [3000], 32, 8, 128, seed=10)
    g = GpuPrefill(spec, q, k, v)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    outs = []
    for start in range(0, 3000, 512):
        end = min(3000, start + 512)
        outs.append(g.run([end], [0, end - start], q=g.q[start:end].contiguous()))
    assert int(g.status.item()) == 0
    assert_parity(torch_to_f64(torch.cat(outs)), ref, "chunked recompute", amended=abs_ref)


def test_bad_lengths_and_ids_are_reported():
    spec, q, k, v, cu = make_case([40, 64], [8, 16], 8, 2, 128, seed=11)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    g = GpuPrefill(spec, q, k, v)
    out = torch_to_f64(g.run([4, 64], cu))           # ctx < q_len for sequence 0
    assert int(g.status.item()) == api.PA_STATUS_BAD_SEQ_LEN
    assert np.isnan(out[:8]).all()                   # rows of the refused sequence untouched
    assert_parity(out[8:], ref[8:], amended=lambda: abs_ref()[8:])
    g.status.zero_()
    t = spec.block_tables.copy()
    t[1, 2] = spec.num_blocks + 5
    out = torch_to_f64(g.run(spec.seq_lens, cu, tables=torch.from_numpy(t).cuda()))
    assert int(g.status.item()) == api.PA_STATUS_BAD_BLOCK_ID
    assert_parity(out[:8], ref[:8], amended=lambda: abs_ref()[:8])
    # queries at positions 48..63 need block 2 (tokens 32..47): all of sequence 1's rows are zero
    assert (out[8:] == 0).all()


@pytest.mark.parametrize("H,Hkv", [(4, 4), (32, 8)])
def test_long_context_chunks_with_ragged_ends(H, Hkv):
    # chunks whose ends are not multiples of the kernels' 16/64/128-token tiles, contexts
    # that end inside a block, several sequences of very different length in one call
    ctx = [4999, 130, 1031, 64]
    qlens = [517, 130, 7, 1]
    spec, q, k, v, cu = make_case(ctx, qlens, H, Hkv, 128, seed=40 + H)
    g = GpuPrefill(spec, q, k, v)
    out = torch_to_f64(g.run(spec.seq_lens, cu))
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert int(g.status.item()) == 0
    assert_parity(out, ref, f"H{H}/{Hkv}", amended=abs_ref)


def test_large_scores_and_growing_maxima():
    # scale 8 makes the running row maximum jump by far more than 2^8 between steps
    spec, q, k, v, cu = make_case([700], [300], 8, 2, 128, seed=50)
    g = GpuPrefill(spec, q, k, v)
    spec.scale = np.float32(8.0)
    out = torch_to_f64(g.run(spec.seq_lens, cu))
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, 8.0)
    # the softmax is nearly one-hot here, so outputs are single V rows, some of magnitude 2-4:
    # the case the amended bound of assert_parity is written for
    assert_parity(out, ref, "scale 8", amended=abs_ref)


def test_large_chunk_takes_the_two_tile_kernel():
    # (2300 / 64 + 2) * 8 KV heads = 296 CTAs of two row tiles fill two rounds of 148 SMs: two
    # softmax warpgroups share the K/V stages; the second sequence ends in a half-used pair
    spec, q, k, v, cu = make_case([2100, 1201], [1500, 800], 32, 8, 128, seed=60)
    g = GpuPrefill(spec, q, k, v)
    out = torch_to_f64(g.run(spec.seq_lens, cu))
    assert api.pa_prefill_last_launch() == (2, 0, 1)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert int(g.status.item()) == 0
    assert_parity(out, ref, "two tiles per CTA", amended=abs_ref)


# ---- KV range split over CTAs (pa_prefill_split) --------------------------------------------

@pytest.mark.parametrize("H,Hkv,D", [(8, 8, 64), (6, 2, 64), (10, 2, 128), (16, 8, 256), (4, 1, 256)])
def test_kv_split_other_head_dims_and_group_sizes(H, Hkv, D):
    # head_dim 64 and 256, and group sizes that do not divide 128 (idle rows in every tile)
    ctx = [2999, 130, 1031, 64]
    qlens = [300, 130, 7, 1]
    spec, q, k, v, cu = make_case(ctx, qlens, H, Hkv, D, seed=90 + H + D)
    split = 512
    max_splits = -(-spec.block_tables.shape[1] * 16 // split)
    g = GpuPrefill(spec, q, k, v, max_splits=max_splits)
    out = torch_to_f64(g.run(spec.seq_lens, cu, split=split))
    tiles, tok, cap = api.pa_prefill_last_launch()
    assert tiles == (1 if D == 256 else tiles) and tiles in (1, 2) and tok == split and cap == max_splits
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert int(g.status.item()) == 0
    assert_parity(out, ref, f"H{H}/{Hkv} D{D} split", amended=abs_ref)


@pytest.mark.parametrize("H,Hkv", [(4, 4), (32, 8), (16, 1)])
@pytest.mark.parametrize("split", [64, 192, 1024])
def test_forced_kv_split_matches_oracle(H, Hkv, split):
    # contexts that end inside a block and inside a split, tiles whose last rows see fewer
    # splits than the sequence has, a sequence that fits one split (written directly), an
    # empty chunk
    ctx = [4999, 130, 1031, 64, 300]
    qlens = [517, 130, 7, 1, 0]
    spec, q, k, v, cu = make_case(ctx, qlens, H, Hkv, 128, seed=70 + H)
    max_splits = -(-spec.block_tables.shape[1] * 16 // split)
    g = GpuPrefill(spec, q, k, v, max_splits=max_splits)
    out = g.run(spec.seq_lens, cu, split=split)
    tiles, tok, cap = api.pa_prefill_last_launch()
    assert tiles in (1, 2) and tok == split and cap == max_splits
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert int(g.status.item()) == 0
    assert_parity(torch_to_f64(out), ref, f"H{H}/{Hkv} split {split}", amended=abs_ref)
    again = g.run(spec.seq_lens, cu, split=split)
    assert torch.equal(out.view(torch.int16), again.view(torch.int16))


@pytest.mark.parametrize("H,Hkv,D", [(9, 3, 64), (3, 3, 128), (5, 1, 256)])
def test_forced_split_with_odd_head_count_and_odd_token_count(H, Hkv, D):
    # 513 query tokens x an odd head count x 3 splits: an odd number of (exponent, sum) pairs
    # precedes the partial rows in the workspace, and those rows are stored 16 bytes at a time
    ctx, qlens = [1343], [513]
    spec, q, k, v, cu = make_case(ctx, qlens, H, Hkv, D, seed=17 + H)
    split = 448
    max_splits = -(-spec.block_tables.shape[1] * 16 // split)
    assert max_splits == 3 and (513 * H * max_splits) % 2 == 1
    g = GpuPrefill(spec, q, k, v, max_splits=max_splits)
    out = torch_to_f64(g.run(spec.seq_lens, cu, split=split))
    assert api.pa_prefill_last_launch()[1:] == (split, max_splits)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert int(g.status.item()) == 0
    assert_parity(out, ref, f"H{H}/{Hkv} D{D} odd split", amended=abs_ref)


def test_split_calls_queued_on_one_workspace_keep_their_counts_apart():
    """The units of a split call count themselves in per row group, in counters that live in
    the workspace and carry the call's number.  Chunks of one growing context are queued on one
    workspace without synchronisation (the recomputation pattern), with different split
    lengths, and one chunk is repeated; every chunk's rows must match the oracle."""
    H, Hkv, D = 32, 8, 128
    L, chunk = 2304, 256
    spec, q, k, v, _ = make_case([L], [L], H, Hkv, D, seed=91)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, np.array([0, L], np.int32),
                               spec.scale)
    g = GpuPrefill(spec, q, k, v, max_splits=40)
    g.ws = torch.full((api.pa_prefill_split_workspace_bytes(api.shape_of(g.k, H), 1, chunk, 40) // 4,),
                      float("nan"), dtype=torch.float32, device="cuda")
    out = torch.full_like(g.q, float("nan"))
    again = torch.full_like(g.q[:chunk], float("nan"))
    splits = [0, 64, 512, 0, 128, 320, 64, 0, 1024]
    for i, start in enumerate(range(0, L, chunk)):
        end = start + chunk
        args = (g.k, g.v, g.tables[:, :(end + 15) // 16].contiguous(),
                torch.tensor([end], dtype=torch.int32, device="cuda"),
                torch.tensor([0, chunk], dtype=torch.int32, device="cuda"), spec.scale)
        api.pa_prefill_split(g.q[start:end], *args, out[start:end], g.ws,
                             kv_split_tokens=splits[i], dev_status=g.status)
        if start == 4 * chunk:  # the same chunk once more, into other rows
            api.pa_prefill_split(g.q[start:end], *args, again, g.ws, kv_split_tokens=64,
                                 dev_status=g.status)
    torch.cuda.synchronize()
    assert int(g.status.item()) == 0
    assert_parity(torch_to_f64(out), ref, "queued split chunks", amended=abs_ref)
    assert_parity(torch_to_f64(again), ref[4 * chunk:5 * chunk], "repeated chunk",
                  amended=lambda: abs_ref()[4 * chunk:5 * chunk])


def test_kv_split_with_two_tiles_per_cta():
    # enough query tokens for two row tiles per CTA; queries in the middle of the context, so
    # the first tiles end before the last splits begin
    spec, q, k, v, cu = make_case([2600, 1111], [1500, 900], 32, 8, 128, seed=80)
    split = 512
    max_splits = -(-spec.block_tables.shape[1] * 16 // split)
    g = GpuPrefill(spec, q, k, v, max_splits=max_splits)
    out = torch_to_f64(g.run(spec.seq_lens, cu, split=split))
    assert api.pa_prefill_last_launch() == (2, split, max_splits)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert int(g.status.item()) == 0
    assert_parity(out, ref, "split, two tiles per CTA", amended=abs_ref)


def test_library_chosen_split_on_a_recompute_chunk():
    # one long victim, the last 256 tokens of a 6000-token context: 16 tiles for 148 SMs, so
    # the library splits the KV range by itself once the workspace allows it
    spec, q, k, v, cu = make_case([6000], [256], 8, 2, 128, seed=81)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    g = GpuPrefill(spec, q, k, v, max_splits=16)
    out = torch_to_f64(g.run(spec.seq_lens, cu, split=0))
    tiles, tok, cap = api.pa_prefill_last_launch()
    assert tok > 0 and 1 < cap <= 16, (tiles, tok, cap)
    assert_parity(out, ref, "library-chosen split", amended=abs_ref)
    # the same call with a workspace that holds no partial rows runs unsplit
    g1 = GpuPrefill(spec, q, k, v)
    out1 = torch_to_f64(g1.run(spec.seq_lens, cu))
    assert api.pa_prefill_last_launch()[1:] == (0, 1)
    assert_parity(out1, ref, "unsplit", amended=abs_ref)
    assert int(g.status.item()) == 0 and int(g1.status.item()) == 0
    # never split on request
    g.run(spec.seq_lens, cu, split=-1)
    assert api.pa_prefill_last_launch()[1:] == (0, 1)


def test_kv_split_errors():
    spec, q, k, v, cu = make_case([2000, 640], [64, 640], 8, 2, 128, seed=82)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    g = GpuPrefill(spec, q, k, v, max_splits=2)
    with pytest.raises(api.PagedKVError) as e:       # 2000 tokens in 256-token splits: 8 rows
        g.run(spec.seq_lens, cu, split=256)
    assert e.value.code == api.ERR["WORKSPACE"]
    g = GpuPrefill(spec, q, k, v, max_splits=8)
    t = spec.block_tables.copy()
    t[0, 40] = spec.num_blocks + 3                   # tokens 640..655 of sequence 0: split 2
    out = torch_to_f64(g.run(spec.seq_lens, cu, tables=torch.from_numpy(t).cuda(), split=256))
    assert int(g.status.item()) == api.PA_STATUS_BAD_BLOCK_ID
    assert (out[:64] == 0).all()                     # every query of sequence 0 sees block 40
    assert_parity(out[64:], ref[64:], amended=lambda: abs_ref()[64:])
    g.status.zero_()
    out = torch_to_f64(g.run([2000, 600], cu, split=256))   # ctx < q_len for sequence 1
    assert int(g.status.item()) == api.PA_STATUS_BAD_SEQ_LEN
    assert np.isnan(out[64:]).all()
    assert_parity(out[:64], ref[:64], amended=lambda: abs_ref()[:64])


@pytest.mark.parametrize("scale", [0.0, -0.25])
@pytest.mark.parametrize("H,Hkv,D", [(8, 2, 128), (8, 8, 64), (4, 1, 256)])
def test_zero_and_negative_scale(scale, H, Hkv, D):
    # scale 0: every query is the mean of the V rows it may see; a negative scale turns the
    # order of the scores around (the kernel's raw-score maximum shortcut needs scale > 0)
    spec, q, k, v, cu = make_case([300, 64, 17], [300, 10, 17], H, Hkv, D, seed=120)
    g = GpuPrefill(spec, q, k, v)
    spec.scale = np.float32(scale)
    out = torch_to_f64(g.run(spec.seq_lens, cu))
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, scale)
    assert int(g.status.item()) == 0
    assert_parity(out, ref, f"scale {scale}", amended=abs_ref)
    if scale == 0.0:   # closed form, independent of the oracle: running mean of V
        from helpers import bits_to_torch
        tab = spec.block_tables[2]
        vv = bits_to_torch(v).float().cpu().numpy()                      # [NB, Hkv, 16, D]
        rows = np.stack([vv[tab[t // 16], :, t % 16] for t in range(17)])    # [17, Hkv, D]
        mean = np.cumsum(rows, axis=0) / np.arange(1, 18)[:, None, None]
        got = out[int(cu[2]):].reshape(17, Hkv, H // Hkv, D)
        assert np.abs(got - mean[:, :, None, :]).max() <= 1e-2


@pytest.mark.parametrize("n_seq", [32, 33, 70])
def test_batches_around_32_sequences(n_seq):
    # up to 32 sequences the attention CTAs plan for themselves; beyond that a plan kernel runs
    rng = np.random.default_rng(n_seq)
    ctx = [int(x) for x in rng.integers(1, 200, n_seq)]
    qlens = [int(rng.integers(0, c + 1)) for c in ctx]
    qlens[0] = max(qlens[0], 1)
    spec, q, k, v, cu = make_case(ctx, qlens, 8, 2, 128, seed=200 + n_seq)
    g = GpuPrefill(spec, q, k, v)
    n0 = api.pa_launch_count()
    out = torch_to_f64(g.run(spec.seq_lens, cu))
    assert api.pa_launch_count() - n0 == (1 if n_seq <= 32 else 2)
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert int(g.status.item()) == 0
    assert_parity(out, ref, f"{n_seq} sequences", amended=abs_ref)
    # and a refused sequence is reported either way
    bad_ctx = spec.seq_lens.copy()
    bad_ctx[n_seq - 1] = -3
    g.run(bad_ctx, cu)
    assert int(g.status.item()) == api.PA_STATUS_BAD_SEQ_LEN
