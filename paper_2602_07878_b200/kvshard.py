"""KV-head sharding of the decode and swap path over tensor-parallel ranks (Section 6.4: TP 2/4/8).

Rank r of R holds KV heads [r * Hkv / R, (r + 1) * Hkv / R) of every block and the query heads
of their groups.  The path has no exchange step in this mode: every rank runs the library's
calls on its own heads and the collective of a tensor-parallel layer (the all-reduce after the
output projection) lies outside it.  This module is index arithmetic and argument marshalling
only; the kernels are the library's.

An engine with one pool per GPU passes that pool and its own [B, H / R, D] tensors and needs
nothing from here.  `views` serves the other case -- batch-wide tensors of which a rank owns a
slice of heads (one GPU standing in for several, or a fused projection output): the slices are
strided views, which `api.pa_decode` forwards to `pa_decode_strided` and the swaps take through
the pool strides, so nothing is copied.
"""
from __future__ import annotations

from typing import Callable, Tuple

from . import api


def head_range(rank: int, world: int, num_q_heads: int, num_kv_heads: int) -> Tuple[slice, slice]:
    """(query heads, KV heads) owned by `rank`.  KV heads are split evenly (world must divide
    their number: a KV head is never shared by two ranks) and query heads follow their group."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("rank outside the group")
    if num_kv_heads % world or num_q_heads % num_kv_heads:
        raise ValueError("the ranks must divide the KV heads, the KV heads the query heads")
    per = num_kv_heads // world
    g = num_q_heads // num_kv_heads
    return slice(rank * per * g, (rank + 1) * per * g), slice(rank * per, (rank + 1) * per)


def views(rank: int, world: int, q, k_cache, v_cache, out=None):
    """This rank's views of q [B, H, D], of caches [..., NB, Hkv, bs, D] (one layer or a pool of
    layers) and of out [B, H, D]: slices along the head axes, no copies."""
    num_q_heads, num_kv_heads = q.shape[1], k_cache.shape[-3]
    qs, ks = head_range(rank, world, num_q_heads, num_kv_heads)
    k_r, v_r = k_cache[..., ks, :, :], v_cache[..., ks, :, :]
    return q[:, qs], k_r, v_r, (None if out is None else out[:, qs])


def decode(rank: int, world: int, q, k_cache, v_cache, block_tables, seq_lens, scale, out,
           workspace, *, decode_fn: Callable = api.pa_decode, **kw):
    """One decode step of `rank` on its heads of batch-wide tensors; writes out[:, its heads]."""
    q_r, k_r, v_r, out_r = views(rank, world, q, k_cache, v_cache, out)
    decode_fn(q_r, k_r, v_r, block_tables, seq_lens, scale, out_r, workspace, **kw)
    return out_r


def workspace_bytes(world: int, k_cache, num_q_heads: int, max_batch: int, max_total_tokens: int,
                    partition_tokens: int = 0) -> int:
    """Workspace one rank needs (every rank has the same head counts)."""
    _, ks = head_range(0, world, num_q_heads, k_cache.shape[-3])
    shape = api.shape_of(k_cache[..., ks, :, :], num_q_heads // world)
    return api.pa_workspace_bytes(shape, max_batch, max_total_tokens, partition_tokens)
