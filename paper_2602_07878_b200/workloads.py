"""Seeded synthetic inputs for paged-attention decode and KV-block swaps.

This module only *draws inputs*: context lengths, block tables, pool occupancy and
bf16 bit patterns.  It holds none of the attention or copy arithmetic, so both the
CPU oracle's tests and the CUDA path's tests may build their inputs from it.

Values.  Every tensor element is a pure function of (stream seed, flat element index):
a 32-bit integer mix of the index selects one of 65536 entries of a table that holds
the standard-normal quantiles at (i + 0.5) / 65536 rounded to bf16.  The draw is
therefore N(0,1) up to that quantisation, needs integer arithmetic only, and gives the
same bits from numpy on the host and from torch integer ops on a device, for any
index, without materialising anything else.  That is what lets a 100 GB pool be filled
on the device while a CPU checker regenerates just the blocks it wants to look at.

Shapes.  The five workloads mirror a serving engine whose paged KV pool is kept close
to full by a mix of short conversations and a few near-limit contexts (Section 5 of
the paper describes the regime: pool usage pinned at 97.5-100 %, prompts of about
500, 1-2 K and near-limit tokens).  They stand in for the paper's Alpaca / ShareGPT /
BurstGPT traffic, which enters the decode step only through these shapes.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np

BF16_NAN_BITS = 0x7FC1          # a quiet NaN pattern used to poison unused slots
TABLE_POISON = (-1, 0x7FFFFFFF)  # written into block-table entries past a sequence's end

_M32 = np.uint64(0xFFFFFFFF)
_BASE_SEED = 0x26020787


# --------------------------------------------------------------------------------------
# bf16 helpers (bit-level only)
# --------------------------------------------------------------------------------------
def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round finite float values to bf16 (nearest even), returned as uint16 bit patterns."""
    b = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))
    return (b >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


_TABLE: Optional[np.ndarray] = None


def normal_table() -> np.ndarray:
    """uint16[65536]: bf16 bits of the N(0,1) quantile at (i + 0.5) / 65536."""
    global _TABLE
    if _TABLE is None:
        from scipy.special import ndtri

        p = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
        _TABLE = f64_to_bf16_bits(ndtri(p))
    return _TABLE


# --------------------------------------------------------------------------------------
# counter hash: numpy and torch versions of the same integer function
# --------------------------------------------------------------------------------------
def _mix32_np(x: np.ndarray) -> np.ndarray:
    x = x ^ (x >> np.uint64(16))
    x = (x * np.uint64(0x85EBCA6B)) & _M32
    x = x ^ (x >> np.uint64(13))
    x = (x * np.uint64(0xC2B2AE35)) & _M32
    x = x ^ (x >> np.uint64(16))
    return x


def hash16_np(idx: np.ndarray, seed: int) -> np.ndarray:
    """16-bit hash of 64-bit counters `idx` under a 32-bit stream seed (numpy)."""
    idx = np.asarray(idx).astype(np.uint64)
    lo = idx & _M32
    hi = idx >> np.uint64(32)
    s = _mix32_np((hi + np.uint64(seed & 0xFFFFFFFF)) & _M32)
    return (_mix32_np(lo ^ s) & np.uint64(0xFFFF)).astype(np.int64)


def _mix32_u32(x: np.ndarray) -> np.ndarray:
    """murmur-style 32-bit finaliser on a uint32 array, in place (products wrap mod 2^32)."""
    x ^= x >> np.uint32(16)
    x *= np.uint32(0x85EBCA6B)
    x ^= x >> np.uint32(13)
    x *= np.uint32(0xC2B2AE35)
    x ^= x >> np.uint32(16)
    return x


def normal_bf16_np(start: int, count: int, seed: int) -> np.ndarray:
    """bf16 bits (uint16[count]) of stream `seed` at flat indices start .. start+count-1.

    Same function as `hash16_np` + table lookup, evaluated in uint32 arithmetic on pieces
    that do not cross a multiple of 2^32 (so the high word is a scalar per piece)."""
    out = np.empty(count, dtype=np.uint16)
    tab = normal_table()
    step = 1 << 22
    o = 0
    while o < count:
        s0 = start + o
        n = min(step, count - o, (1 << 32) - (s0 & 0xFFFFFFFF))
        hi = s0 >> 32
        sh = int(_mix32_np(np.array([(hi + (seed & 0xFFFFFFFF)) & 0xFFFFFFFF], np.uint64))[0])
        x = np.arange(s0 & 0xFFFFFFFF, (s0 & 0xFFFFFFFF) + n, dtype=np.uint64).astype(np.uint32)
        x ^= np.uint32(sh)
        _mix32_u32(x)
        x &= np.uint32(0xFFFF)
        np.take(tab, x, out=out[o:o + n])
        o += n
    return out


def _mix32_t(x):
    m = 0xFFFFFFFF
    x = x ^ (x >> 16)
    x = (x * 0x85EBCA6B) & m
    x = x ^ (x >> 13)
    x = (x * 0xC2B2AE35) & m
    x = x ^ (x >> 16)
    return x


def normal_bf16_torch(start: int, count: int, seed: int, device, out=None):
    """Same stream as `normal_bf16_np`, produced with torch integer ops on `device`.

    Returns (or fills) a torch.bfloat16 tensor of `count` elements.  Work is chunked so
    that the int64 temporaries stay below about 2 GB.
    """
    import torch

    if out is None:
        out = torch.empty(count, dtype=torch.bfloat16, device=device)
    flat = out.view(-1).view(torch.int16)
    tab = torch.from_numpy(normal_table().view(np.int16).copy()).to(device)
    step = 1 << 25
    for o in range(0, count, step):
        n = min(step, count - o)
        idx = torch.arange(start + o, start + o + n, dtype=torch.int64, device=device)
        lo = idx & 0xFFFFFFFF
        hi = idx >> 32
        s = _mix32_t((hi + (seed & 0xFFFFFFFF)) & 0xFFFFFFFF)
        h = _mix32_t(lo ^ s) & 0xFFFF
        flat[o:o + n] = tab[h]
        del idx, lo, hi, s, h
    return out


# --------------------------------------------------------------------------------------
# workload description
# --------------------------------------------------------------------------------------
@dataclasses.dataclass
class DecodeSpec:
    """Shape, lengths and block tables of one decode batch (no tensor values)."""

    name: str
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    num_blocks: int                 # physical pool size NB
    seq_lens: np.ndarray            # int32[B]
    block_tables: np.ndarray        # int32[B, max_blocks], poisoned past each row's end
    scale: np.float32
    seed: int
    free_blocks: np.ndarray         # int32[...] physical ids not referenced by any table
    num_layers: int = 1

    @property
    def batch(self) -> int:
        return int(self.seq_lens.shape[0])

    @property
    def max_blocks(self) -> int:
        return int(self.block_tables.shape[1])

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def block_elems(self) -> int:
        """Elements of one block of one of K or V for one layer: Hkv * bs * D."""
        return self.num_kv_heads * self.block_size * self.head_dim

    @property
    def total_tokens(self) -> int:
        return int(self.seq_lens.astype(np.int64).sum())

    def blocks_of(self, b: int) -> np.ndarray:
        nb = (int(self.seq_lens[b]) + self.block_size - 1) // self.block_size
        return self.block_tables[b, :nb].copy()

    def kv_bytes(self) -> int:
        """Bytes of K and V the attention step must read: sum_b L_b * 2 * Hkv * D * 2."""
        return self.total_tokens * 2 * self.num_kv_heads * self.head_dim * 2

    def algorithmic_bytes(self) -> int:
        """KV bytes + q + out + the block-table entries and lengths actually needed."""
        bs = self.block_size
        nblk = int(((self.seq_lens.astype(np.int64) + bs - 1) // bs).sum())
        qo = 2 * self.batch * self.num_q_heads * self.head_dim * 2
        return self.kv_bytes() + qo + 4 * nblk + 4 * self.batch

    # seeds of the three value streams
    @property
    def seed_q(self) -> int:
        return (self.seed * 4 + 1) & 0xFFFFFFFF

    @property
    def seed_k(self) -> int:
        return (self.seed * 4 + 2) & 0xFFFFFFFF

    @property
    def seed_v(self) -> int:
        return (self.seed * 4 + 3) & 0xFFFFFFFF


def _build_tables(seq_lens: np.ndarray, block_size: int, num_blocks: int,
                  rng: np.random.Generator, max_blocks: Optional[int] = None):
    """Deal the first `alloc` ids of a seeded permutation of the pool to the sequences.

    A random permutation leaves consecutive logical blocks of a sequence far apart in
    the pool (a fragmented allocator state).  Entries past a row's end are poisoned.
    """
    nb = (seq_lens.astype(np.int64) + block_size - 1) // block_size
    alloc = int(nb.sum())
    if alloc > num_blocks:
        raise ValueError(f"{alloc} blocks needed, pool has {num_blocks}")
    perm = rng.permutation(num_blocks).astype(np.int32)
    mb = int(max_blocks if max_blocks is not None else max(1, nb.max(initial=0)))
    tables = np.empty((len(seq_lens), mb), dtype=np.int32)
    tables[:, 0::2] = TABLE_POISON[0]
    tables[:, 1::2] = TABLE_POISON[1]
    o = 0
    for b, n in enumerate(nb):
        tables[b, :n] = perm[o:o + n]
        o += int(n)
    return tables, perm[alloc:].copy()


def _pool_for_occupancy(seq_lens, block_size, occupancy):
    nb = int(((seq_lens.astype(np.int64) + block_size - 1) // block_size).sum())
    return max(1, int(math.ceil(nb / occupancy)))   # a pool has at least one block


def make_spec(name: str, *, seq_lens, num_q_heads, num_kv_heads, head_dim, block_size=16,
              num_blocks=None, occupancy=None, seed=0, max_blocks=None,
              num_layers=1) -> DecodeSpec:
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    rng = np.random.Generator(np.random.PCG64(seed))
    if num_blocks is None:
        num_blocks = _pool_for_occupancy(seq_lens, block_size, occupancy)
    tables, free = _build_tables(seq_lens, block_size, num_blocks, rng, max_blocks)
    return DecodeSpec(name=name, num_q_heads=num_q_heads, num_kv_heads=num_kv_heads,
                      head_dim=head_dim, block_size=block_size, num_blocks=num_blocks,
                      seq_lens=seq_lens, block_tables=tables,
                      scale=np.float32(1.0 / math.sqrt(head_dim)), seed=seed,
                      free_blocks=free, num_layers=num_layers)


def config_spec(index: int, scale_down: int = 1) -> DecodeSpec:
    """The five workloads (index 1..5).  `scale_down` > 1 divides the batch (and, for
    workload 4, the pool) so that CPU tests can use the same recipe at a smaller size."""
    seed = _BASE_SEED + index
    rng = np.random.Generator(np.random.PCG64(seed ^ 0x5EED))
    if index == 1:
        return make_spec("cfg1_tiny_mha", seq_lens=[17, 64, 100, 256], num_q_heads=8,
                         num_kv_heads=8, head_dim=64, num_blocks=40, seed=seed)
    if index == 2:
        B = max(1, 64 // scale_down)
        lens = rng.integers(128, 2048, size=B, endpoint=True)
        return make_spec("cfg2_llama2_7b_mha", seq_lens=lens, num_q_heads=32,
                         num_kv_heads=32, head_dim=128, occupancy=0.90, seed=seed)
    if index == 3:
        n_long = max(1, 8 // scale_down)
        n_body = max(1, 248 // scale_down)
        body = np.clip(np.rint(np.exp(math.log(300.0) + 1.0 * rng.standard_normal(n_body))),
                       16, 4096)
        lens = np.concatenate([np.full(n_long, 32768), body]).astype(np.int64)
        rng.shuffle(lens)
        return make_spec("cfg3_fullpool_mixed_gqa", seq_lens=lens, num_q_heads=32,
                         num_kv_heads=8, head_dim=128, occupancy=0.99, seed=seed)
    if index == 4:
        pool = max(64, 60000 // scale_down)
        target = int(pool * 0.98)
        n_long = max(1, 8 // scale_down)
        lens = [32768] * n_long
        used = n_long * (32768 // 16)
        if used > target:
            lens, used = [], 0
        while True:
            L = int(np.clip(np.rint(np.exp(math.log(300.0) + rng.standard_normal())), 16, 4096))
            nb = (L + 15) // 16
            if used + nb > target:
                rest = target - used
                if rest > 0:
                    lens.append(rest * 16)
                break
            lens.append(L)
            used += nb
        lens = np.asarray(lens, dtype=np.int64)
        rng.shuffle(lens)
        return make_spec("cfg4_swap_churn", seq_lens=lens, num_q_heads=32, num_kv_heads=8,
                         head_dim=128, num_blocks=pool, seed=seed, num_layers=32)
    if index == 5:
        B = max(1, 128 // scale_down)
        lens = rng.integers(1024, 16384, size=B, endpoint=True)
        return make_spec("cfg5_70b_gqa", seq_lens=lens, num_q_heads=64, num_kv_heads=8,
                         head_dim=128, occupancy=0.95, seed=seed)
    raise ValueError("workload index must be 1..5")


# --------------------------------------------------------------------------------------
# tensor values for a spec
# --------------------------------------------------------------------------------------
def pool_block_np(spec: DecodeSpec, which: str, block_ids, layer: int = 0) -> np.ndarray:
    """uint16[len(ids), Hkv, bs, D]: bf16 bits of the listed physical blocks of the K
    ('k') or V ('v') pool of one layer, regenerated from the counter stream."""
    seed = spec.seed_k if which == "k" else spec.seed_v
    be = spec.block_elems
    out = np.empty((len(block_ids), be), dtype=np.uint16)
    for i, p in enumerate(np.asarray(block_ids, dtype=np.int64)):
        start = (layer * spec.num_blocks + int(p)) * be
        out[i] = normal_bf16_np(start, be, seed)
    return out.reshape(len(block_ids), spec.num_kv_heads, spec.block_size, spec.head_dim)


def q_np(spec: DecodeSpec) -> np.ndarray:
    n = spec.batch * spec.num_q_heads * spec.head_dim
    return normal_bf16_np(0, n, spec.seed_q).reshape(spec.batch, spec.num_q_heads, spec.head_dim)


def pools_np(spec: DecodeSpec, layer: int = 0, poison_tails: bool = True):
    """Full K and V pools of one layer as uint16[NB, Hkv, bs, D] (host; small specs only)."""
    be = spec.block_elems
    n = spec.num_blocks * be
    shape = (spec.num_blocks, spec.num_kv_heads, spec.block_size, spec.head_dim)
    k = normal_bf16_np(layer * n, n, spec.seed_k).reshape(shape)
    v = normal_bf16_np(layer * n, n, spec.seed_v).reshape(shape)
    if poison_tails:
        for blk, slot in tail_slots(spec):
            k[blk, :, slot:, :] = BF16_NAN_BITS
            v[blk, :, slot:, :] = BF16_NAN_BITS
    return k, v


def tail_slots(spec: DecodeSpec):
    """(physical block, first unused slot) of every sequence whose last block is partial."""
    out = []
    bs = spec.block_size
    for b in range(spec.batch):
        L = int(spec.seq_lens[b])
        if L > 0 and L % bs:
            out.append((int(spec.block_tables[b, (L - 1) // bs]), L % bs))
    return out


def pools_torch(spec: DecodeSpec, device, layer: int = 0, poison_tails: bool = True):
    """Device K and V pools (torch.bfloat16 [NB, Hkv, bs, D]) with the same bits as `pools_np`."""
    import torch

    n = spec.num_blocks * spec.block_elems
    shape = (spec.num_blocks, spec.num_kv_heads, spec.block_size, spec.head_dim)
    k = normal_bf16_torch(layer * n, n, spec.seed_k, device).view(shape)
    v = normal_bf16_torch(layer * n, n, spec.seed_v, device).view(shape)
    if poison_tails:
        k16, v16 = k.view(torch.int16), v.view(torch.int16)
        for blk, slot in tail_slots(spec):
            k16[blk, :, slot:, :] = BF16_NAN_BITS      # same bit pattern as the host pools
            v16[blk, :, slot:, :] = BF16_NAN_BITS
    return k, v


def q_torch(spec: DecodeSpec, device):
    n = spec.batch * spec.num_q_heads * spec.head_dim
    return normal_bf16_torch(0, n, spec.seed_q, device).view(
        spec.batch, spec.num_q_heads, spec.head_dim)


# --------------------------------------------------------------------------------------
# eviction sets for the swap workload
# --------------------------------------------------------------------------------------
def pick_victims(spec: DecodeSpec, n_tokens: int, seed: int):
    """Seeded random set of whole sequences totalling about `n_tokens` tokens.

    Returns (sequence indices, their physical block ids concatenated in logical order,
    the same number of distinct free ids to restore into).  The last victim's block list
    is truncated so that the total is n_tokens rounded up to whole blocks.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    order = rng.permutation(spec.batch)
    want = (n_tokens + spec.block_size - 1) // spec.block_size
    seqs, ids = [], []
    got = 0
    for b in order:
        blk = spec.blocks_of(int(b))
        if len(blk) == 0:
            continue
        take = min(len(blk), want - got)
        seqs.append(int(b))
        ids.append(blk[:take])
        got += take
        if got >= want:
            break
    ids = np.concatenate(ids).astype(np.int32) if ids else np.zeros(0, np.int32)
    free = spec.free_blocks
    if len(free) < len(ids):
        # a nearly full pool has fewer free blocks than victims: reuse the victims' own
        # ids (they are free after the swap-out) in a shuffled order, after the free ones
        extra = rng.permutation(ids)[: len(ids) - len(free)]
        dest = np.concatenate([rng.permutation(free), extra]).astype(np.int32)
    else:
        dest = rng.permutation(free)[: len(ids)].astype(np.int32)
    return seqs, ids, dest
