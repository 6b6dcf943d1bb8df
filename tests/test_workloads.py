"""The seeded input generators: same bits from numpy and torch, N(0,1)-like values, and
the five workload recipes (lengths, occupancy, fragmentation, poison)."""
import numpy as np
import torch

from paper_2602_07878_b200 import workloads as wl


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.5, 0.0, 1e-3])
    bits = wl.f64_to_bf16_bits(x)
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy()
    assert (bits.view(np.int16) == ref).all()
    assert (wl.bf16_bits_to_f64(bits)[:2] == 1.0).all()       # tie to even


def test_numpy_and_torch_streams_agree():
    for start in (0, 12345, (1 << 32) - 100, (1 << 36) + 7):
        a = wl.normal_bf16_np(start, 5000, 99)
        b = wl.normal_bf16_torch(start, 5000, 99, "cpu").view(torch.int16).numpy()
        assert (a.view(np.int16) == b).all()


def test_stream_is_standard_normal_like():
    x = wl.bf16_bits_to_f64(wl.normal_bf16_np(0, 1 << 20, 5))
    assert abs(x.mean()) < 5e-3 and abs(x.std() - 1.0) < 5e-3
    assert np.abs(x).max() < 4.5
    y = wl.bf16_bits_to_f64(wl.normal_bf16_np(0, 1 << 20, 6))
    assert abs(np.corrcoef(x, y)[0, 1]) < 5e-3
    assert abs(np.corrcoef(x[:-1], x[1:])[0, 1]) < 5e-3


def test_cfg1_shape():
    s = wl.config_spec(1)
    assert list(s.seq_lens) == [17, 64, 100, 256] and s.num_blocks == 40
    assert s.num_q_heads == 8 and s.num_kv_heads == 8 and s.head_dim == 64
    used = np.concatenate([s.blocks_of(b) for b in range(4)])
    assert len(used) == 29 and len(set(used.tolist())) == 29
    assert len(s.free_blocks) == 11 and not set(s.free_blocks.tolist()) & set(used.tolist())
    assert s.total_tokens == 437 and s.kv_bytes() == 437 * 2 * 8 * 64 * 2


def test_full_size_recipes():
    s2, s3, s5 = wl.config_spec(2), wl.config_spec(3), wl.config_spec(5)
    assert s2.batch == 64 and s2.seq_lens.min() >= 128 and s2.seq_lens.max() <= 2048
    assert s3.batch == 256 and (s3.seq_lens == 32768).sum() == 8
    body = np.sort(s3.seq_lens)[:248]
    assert body.min() >= 16 and body.max() <= 4096 and 200 < np.median(body) < 450
    assert s5.batch == 128 and s5.seq_lens.min() >= 1024 and s5.seq_lens.max() <= 16384
    for s, occ in ((s2, 0.90), (s3, 0.99), (s5, 0.95)):
        alloc = s.num_blocks - len(s.free_blocks)
        assert abs(alloc / s.num_blocks - occ) < 2e-3
        # fragmented: consecutive logical blocks are almost never physically adjacent
        b = int(np.argmax(s.seq_lens))
        ids = s.blocks_of(b).astype(np.int64)
        assert (np.abs(np.diff(ids)) == 1).mean() < 0.01
    s4 = wl.config_spec(4)
    assert s4.num_blocks == 60000 and s4.num_layers == 32
    assert s4.num_blocks - len(s4.free_blocks) == 58800


def test_poison_positions():
    s = wl.config_spec(1)
    k, v = wl.pools_np(s)
    tails = dict(wl.tail_slots(s))
    assert len(tails) == 2                    # 17 and 100 are not multiples of 16
    for blk, slot in tails.items():
        assert (k[blk, :, slot:] == wl.BF16_NAN_BITS).all()
        assert (k[blk, :, :slot] != wl.BF16_NAN_BITS).all()
    blk = wl.pool_block_np(s, "k", [3, 17])
    kc, _ = wl.pools_np(s, poison_tails=False)
    assert (blk == kc[[3, 17]]).all()


def test_pick_victims_totals_and_distinct_destinations():
    s = wl.config_spec(4, scale_down=20)
    for n_tok in (1024, 4096):
        seqs, ids, dest = wl.pick_victims(s, n_tok, seed=1)
        assert len(ids) == n_tok // 16 and len(dest) == len(ids)
        assert len(set(dest.tolist())) == len(dest)
        assert len(set(ids.tolist())) == len(ids)
