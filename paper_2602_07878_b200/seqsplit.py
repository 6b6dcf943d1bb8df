"""Sequence-split decode over several ranks: host-side sharding and the one exchange step.

Every rank keeps a contiguous run of each sequence's logical blocks in its own pool, attends
over that slice with `pa_decode_partial`, all-gathers the partial records (B*H*(D+2) floats
per rank) and merges them with `pa_merge_partials`.  Nothing else crosses the link.  The
kernels are the library's; this module only slices tables and moves the records.
"""
from __future__ import annotations

from typing import Callable, Optional, Tuple

import numpy as np
import torch
import torch.distributed as dist

from . import api


def shard_bounds(num_blocks: np.ndarray, rank: int, world: int) -> Tuple[np.ndarray, np.ndarray]:
    """First and one-past-last logical block of every sequence held by `rank`: an even split
    by blocks, earlier ranks holding the earlier tokens."""
    nb = np.asarray(num_blocks, dtype=np.int64)
    return nb * rank // world, nb * (rank + 1) // world


def shard_context(block_tables: np.ndarray, seq_lens: np.ndarray, rank: int, world: int,
                  block_size: int = 16) -> Tuple[np.ndarray, np.ndarray]:
    """(local block table int32 [B, max_local], local lengths int32 [B]) of `rank`.

    The local table lists the rank's slice of each row of `block_tables` from column 0 on;
    unused entries are -1.  Lengths count the tokens of the slice (only the last slice of a
    sequence can end inside a block)."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the group")
    lens = np.asarray(seq_lens, dtype=np.int64)
    nb = (lens + block_size - 1) // block_size
    lo, hi = shard_bounds(nb, rank, world)
    width = max(1, int((hi - lo).max()) if len(lens) else 1)
    local = np.full((len(lens), width), -1, dtype=np.int32)
    for b in range(len(lens)):
        local[b, : hi[b] - lo[b]] = block_tables[b, lo[b]:hi[b]]
    local_lens = np.clip(lens - lo * block_size, 0, (hi - lo) * block_size).astype(np.int32)
    return local, local_lens


def exchange(part: torch.Tensor, gathered: Optional[torch.Tensor] = None,
             group=None) -> torch.Tensor:
    """All-gather one partial record per rank into [world, n] (rank order)."""
    world = dist.get_world_size(group)
    flat = part.reshape(-1)
    if gathered is None:
        gathered = torch.empty((world, flat.numel()), dtype=part.dtype, device=part.device)
    assert gathered.shape == (world, flat.numel()) and gathered.is_contiguous()
    dist.all_gather_into_tensor(gathered.view(-1), flat, group=group)
    return gathered


def decode(q, k_cache, v_cache, local_tables, local_lens, scale, out, workspace, part,
           gathered=None, group=None, *,
           partial_fn: Callable = api.pa_decode_partial,
           merge_fn: Callable = api.pa_merge_partials, **kw):
    """One sequence-split decode step on this rank: partial attention over the local slice,
    all-gather, merge.  Every rank ends with the full `out` [B,H,D]."""
    B, H, D = q.shape
    partial_fn(q, k_cache, v_cache, local_tables, local_lens, scale, part, workspace, **kw)
    gathered = exchange(part, gathered, group)
    merge_fn(gathered, B * H, D, out)
    return out
