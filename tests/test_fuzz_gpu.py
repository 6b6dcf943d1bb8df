"""Seeded random cases of the three attention entry points against the oracle: random head
layouts, batch sizes and length mixes (zero and one-token sequences, lengths that end on and
off block, partition and tile boundaries), random forced partition / split sizes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from helpers import GpuDecode, assert_parity, bits_to_torch, torch_to_f64

pytestmark = pytest.mark.gpu

LAYOUTS = [(8, 8, 64), (8, 2, 64), (12, 4, 64), (4, 4, 128), (32, 8, 128), (16, 1, 128), (10, 2, 128),
           (6, 6, 128), (8, 2, 256), (16, 8, 256), (3, 1, 256)]
EDGES = [0, 1, 15, 16, 17, 63, 64, 65, 127, 128, 129, 255, 256, 511, 512, 513, 1023, 1024, 1025]


def random_lens(rng, n, hi):
    out = []
    for _ in range(n):
        r = rng.random()
        if r < 0.35:
            out.append(int(rng.choice(EDGES)))
        elif r < 0.85:
            out.append(int(rng.integers(1, 400)))
        else:
            out.append(int(rng.integers(400, hi)))
    return out


@pytest.mark.parametrize("seed", range(24))
def test_random_decode_cases(seed):
    rng = np.random.default_rng(7000 + seed)
    H, Hkv, D = LAYOUTS[int(rng.integers(0, len(LAYOUTS)))]
    lens = random_lens(rng, int(rng.integers(1, 40)), 3000)
    spec = wl.make_spec("fuzz", seq_lens=lens, num_q_heads=H, num_kv_heads=Hkv, head_dim=D,
                        occupancy=float(rng.choice([0.5, 0.9, 1.0])), seed=seed)
    q, (k, v) = wl.q_np(spec), wl.pools_np(spec)
    P = int(rng.choice([0, 0, 64, 128, 256, 512]))
    g = GpuDecode(spec, q, k, v, partition_tokens=P)
    out = torch_to_f64(g.run())
    assert int(g.status.item()) == 0
    ref = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert_parity(out, ref, f"decode seed {seed}: H{H}/{Hkv} D{D} P{P} lens {lens}")


# 60 and 65 are seeds on which one element near 2.2 is rounded to its farther bf16 neighbour
# (error 1.005e-2): the cases behind the spacing rule of assert_parity; 124 did the same under a
# variant of the kernel that summed the rounded weights
@pytest.mark.parametrize("seed", list(range(24)) + [60, 65, 124])
def test_random_prefill_cases(seed):
    rng = np.random.default_rng(8000 + seed)
    H, Hkv, D = LAYOUTS[int(rng.integers(0, len(LAYOUTS)))]
    n = int(rng.integers(1, 7))
    ctx = [max(1, x) for x in random_lens(rng, n, 2500)]
    qlens = [int(rng.choice([0, 1, L, min(L, int(rng.integers(1, 300)))])) for L in ctx]
    if sum(qlens) == 0:
        qlens[0] = 1
    spec = wl.make_spec("fuzz", seq_lens=ctx, num_q_heads=H, num_kv_heads=Hkv, head_dim=D,
                        occupancy=0.9, seed=100 + seed)
    k, v = wl.pools_np(spec)
    cu = np.concatenate([[0], np.cumsum(qlens)]).astype(np.int32)
    q = wl.normal_bf16_np(0, int(cu[-1]) * H * D, 8100 + seed).reshape(int(cu[-1]), H, D)
    split = int(rng.choice([-1, 0, 64, 128, 320, 1024]))
    steps = -(-spec.block_tables.shape[1] * 16 // 64)
    max_splits = 16 if split <= 0 else -(-steps // (-(-split // 64)))
    kd, vd, qd = bits_to_torch(k), bits_to_torch(v), bits_to_torch(q)
    ws = torch.full((api.pa_prefill_split_workspace_bytes(api.shape_of(kd, H), n, int(cu[-1]),
                                                          max_splits) // 4,),
                    float("nan"), dtype=torch.float32, device="cuda")
    out = torch.full_like(qd, float("nan"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.pa_prefill_split(qd, kd, vd, torch.from_numpy(spec.block_tables).cuda(),
                         torch.from_numpy(spec.seq_lens).cuda(), torch.from_numpy(cu).cuda(),
                         spec.scale, out, ws, kv_split_tokens=split, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.pa_prefill(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert_parity(torch_to_f64(out), ref,
                  f"prefill seed {seed}: H{H}/{Hkv} D{D} split {split} ctx {ctx} q {qlens}")
