"""kv_append on the GPU is bit-exact against the append oracle, and a decode step after an
append matches the oracle decoding the grown sequences."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from helpers import GpuDecode, assert_parity, bits_to_torch, torch_to_f64

pytestmark = pytest.mark.gpu


def as_bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("Hkv,D", [(8, 128), (2, 64), (5, 128), (8, 256)])
def test_append_bit_exact_and_nothing_else_changes(Hkv, D):
    lens = np.arange(0, 70, 3)
    spec = wl.make_spec("t", seq_lens=lens, num_q_heads=Hkv, num_kv_heads=Hkv, head_dim=D,
                        occupancy=0.7, seed=Hkv + D)
    k, v = wl.pools_np(spec, poison_tails=False)
    B = spec.batch
    kn = wl.normal_bf16_np(0, B * Hkv * D, 80).reshape(B, Hkv, D)
    vn = wl.normal_bf16_np(0, B * Hkv * D, 81).reshape(B, Hkv, D)
    free = list(spec.free_blocks)
    slots = np.empty(B, np.int64)
    for b in range(B):
        L = int(lens[b])
        if b % 7 == 3:
            slots[b] = -1                                   # padding entry
        elif L % 16 == 0:
            slots[b] = int(free.pop()) * 16                 # needs a fresh block
        else:
            slots[b] = int(spec.block_tables[b, L // 16]) * 16 + L % 16
    kd, vd = bits_to_torch(k), bits_to_torch(v)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.kv_append(kd, vd, bits_to_torch(kn), bits_to_torch(vn), torch.from_numpy(slots).cuda(),
                  dev_status=status)
    torch.cuda.synchronize()
    oracle.kv_append(k, v, kn, vn, slots)
    assert int(status.item()) == 0
    assert (as_bits(kd) == k).all() and (as_bits(vd) == v).all()


def test_append_on_token_major_layout_and_bad_slot():
    spec = wl.make_spec("t", seq_lens=[3, 20], num_q_heads=4, num_kv_heads=4, head_dim=128,
                        num_blocks=6, seed=9)
    k, v = wl.pools_np(spec, poison_tails=False)
    kd = bits_to_torch(k).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vd = bits_to_torch(v).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    kn = wl.normal_bf16_np(0, 2 * 4 * 128, 82).reshape(2, 4, 128)
    vn = wl.normal_bf16_np(0, 2 * 4 * 128, 83).reshape(2, 4, 128)
    slots = np.array([int(spec.block_tables[0, 0]) * 16 + 3, 6 * 16], np.int64)   # 2nd is out of range
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.kv_append(kd, vd, bits_to_torch(kn), bits_to_torch(vn), torch.from_numpy(slots).cuda(),
                  dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == api.PA_STATUS_BAD_BLOCK_ID
    slots[1] = -1
    oracle.kv_append(k, v, kn, vn, slots)
    assert (as_bits(kd) == k).all() and (as_bits(vd) == v).all()


def test_decode_steps_that_grow_sequences_across_block_boundaries():
    """Three decode iterations: append one token per sequence, then attend.  Sequences of
    lengths 15, 16, 31, 47 cross block boundaries on different steps."""
    lens0 = np.array([15, 16, 31, 47, 200], np.int32)
    spec = wl.make_spec("t", seq_lens=lens0 + 3, num_q_heads=8, num_kv_heads=2, head_dim=128,
                        occupancy=0.8, seed=12)              # tables already hold the grown sizes
    k, v = wl.pools_np(spec, poison_tails=False)
    B = spec.batch
    # slots at or beyond each starting length are not written yet: poison them
    for b in range(B):
        for t in range(int(lens0[b]), int(lens0[b]) + 3):
            p, j = int(spec.block_tables[b, t // 16]), t % 16
            k[p, :, j, :] = wl.BF16_NAN_BITS
            v[p, :, j, :] = wl.BF16_NAN_BITS
    q = wl.q_np(spec)
    g = GpuDecode(spec, q, k, v, lens=lens0)
    for step in range(3):
        kn = wl.normal_bf16_np(step * 10000, B * 2 * 128, 90).reshape(B, 2, 128)
        vn = wl.normal_bf16_np(step * 10000, B * 2 * 128, 91).reshape(B, 2, 128)
        pos = lens0 + step
        slots = np.array([int(spec.block_tables[b, pos[b] // 16]) * 16 + pos[b] % 16
                          for b in range(B)], np.int64)
        api.kv_append(g.k, g.v, bits_to_torch(kn), bits_to_torch(vn),
                      torch.from_numpy(slots).cuda())
        oracle.kv_append(k, v, kn, vn, slots)
        lens = (pos + 1).astype(np.int32)
        g.lens.copy_(torch.from_numpy(lens))
        out = torch_to_f64(g.run())
        ref = oracle.pa_decode(q, k, v, spec.block_tables, lens, spec.scale)
        assert_parity(out, ref, f"step {step}")
