"""Seeded random cases of the three attention entry points against the oracle: random head
layouts, batch sizes and length mixes (zero and one-token sequences, lengths that end on and
off block, partition and tile boundaries), random forced partition / split sizes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_07878_b200 import api
from paper_2602_07878_b200 import workloads as wl
from helpers import GpuDecode, assert_parity, bits_to_torch, prefill_ref, torch_to_f64

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


# Thousands of sequences of a few tokens each: their softmax sits on one or two tokens, so
# outputs of magnitude 2 to 5 are common and the rounding of the weights would show.  With
# weights rounded once to bf16, seeds 15, 36 and 78 each had an element off by more than 1e-2.
@pytest.mark.parametrize("seed", [3, 15, 36, 78])
def test_big_batches_of_short_sequences(seed):
    rng = np.random.default_rng(50000 + seed)
    layouts = LAYOUTS + [(16, 1, 64), (32, 2, 128), (16, 1, 256), (64, 8, 128)]
    H, Hkv, D = layouts[int(rng.integers(0, len(layouts)))]
    n = int(rng.integers(900, 3000))
    lens = rng.integers(0, 90, size=n)
    for i in rng.integers(0, n, size=6):
        lens[i] = int(rng.integers(300, 5000))
    spec = wl.make_spec("big", seq_lens=lens, num_q_heads=H, num_kv_heads=Hkv, head_dim=D,
                        occupancy=0.95, seed=seed)
    q, (k, v) = wl.q_np(spec), wl.pools_np(spec)
    P = int(rng.choice([0, 0, 64, 256, 512]))
    g = GpuDecode(spec, q, k, v, partition_tokens=P)
    out = torch_to_f64(g.run())
    assert int(g.status.item()) == 0
    ref = oracle.pa_decode(q, k, v, spec.block_tables, spec.seq_lens, spec.scale)
    assert_parity(out, ref, f"big batch seed {seed}: {n} sequences H{H}/{Hkv} D{D} P{P}")


# 60 and 65 are seeds on which one element near 2.2 is rounded to its farther bf16 neighbour
# (error 1.005e-2): the cases behind the amended bound of assert_parity; 124 did the same under
# a variant of the kernel that summed the rounded weights
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
    ref, abs_ref = prefill_ref(q, k, v, spec.block_tables, spec.seq_lens, cu, spec.scale)
    assert_parity(torch_to_f64(out), ref,
                  f"prefill seed {seed}: H{H}/{Hkv} D{D} split {split} ctx {ctx} q {qlens}",
                  amended=abs_ref)


@pytest.mark.parametrize("seed", range(10))
def test_random_swap_and_append_cases_are_bit_exact(seed):
    rng = np.random.default_rng(9000 + seed)
    layers, Hkv, D = int(rng.integers(1, 6)), int(rng.choice([1, 2, 8])), int(rng.choice([64, 128, 256]))
    NB = int(rng.integers(8, 120))
    n = layers * NB * Hkv * 16 * D
    k = wl.normal_bf16_np(0, n, 9100 + seed).reshape(layers, NB, Hkv, 16, D)
    v = wl.normal_bf16_np(0, n, 9200 + seed).reshape(layers, NB, Hkv, 16, D)
    kd, vd = bits_to_torch(k), bits_to_torch(v)
    if rng.integers(0, 2):   # all layers of a block stored together
        store = torch.empty(NB, layers, 2, Hkv, 16, D, dtype=torch.bfloat16, device="cuda")
        store[:, :, 0], store[:, :, 1] = kd.permute(1, 0, 2, 3, 4), vd.permute(1, 0, 2, 3, 4)
        kd, vd = store[:, :, 0].permute(1, 0, 2, 3, 4), store[:, :, 1].permute(1, 0, 2, 3, 4)
    as_bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    m = int(rng.integers(1, NB // 2 + 1))
    perm = rng.permutation(NB)
    src, dst = perm[:m].astype(np.int32), perm[m:2 * m].astype(np.int32)
    bb = api.kv_block_bytes(kd, vd)
    host = torch.zeros(m * bb, dtype=torch.uint8).pin_memory()
    staging = (torch.empty(int(rng.integers(1, m + 1)) * bb, dtype=torch.uint8, device="cuda")
               if rng.integers(0, 2) else None)
    api.kv_swap_out(kd, vd, src, host, staging)
    torch.cuda.synchronize()
    image = oracle.swap_out(k, v, src)
    assert (host.numpy().view(np.uint16) == image.reshape(-1)).all()
    api.kv_swap_in(kd, vd, host, dst, staging)
    torch.cuda.synchronize()
    oracle.swap_in(k, v, image, dst)
    assert (as_bits(kd) == k).all() and (as_bits(vd) == v).all()
    # append: random tokens into random distinct slots of one layer, some entries skipped
    layer = int(rng.integers(0, layers))
    B = int(rng.integers(1, 50))
    slots = rng.permutation(NB * 16)[:B].astype(np.int64)
    slots[rng.random(B) < 0.2] = -1
    kn = wl.normal_bf16_np(0, B * Hkv * D, 9300 + seed).reshape(B, Hkv, D)
    vn = wl.normal_bf16_np(0, B * Hkv * D, 9400 + seed).reshape(B, Hkv, D)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.kv_append(kd[layer], vd[layer], bits_to_torch(kn), bits_to_torch(vn),
                  torch.from_numpy(slots).cuda(), dev_status=status)
    torch.cuda.synchronize()
    oracle.kv_append(k[layer], v[layer], kn, vn, slots)
    assert int(status.item()) == 0
    assert (as_bits(kd) == k).all() and (as_bits(vd) == v).all()
