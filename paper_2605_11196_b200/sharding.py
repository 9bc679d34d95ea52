"""Splitting one [B,H,T,d] problem over data-parallel ranks.

The (batch, head) units of the scan are independent (Section 3.3 states the recurrence per
head), so N ranks share a problem by taking contiguous ranges of the batch index: a rank's
q, k, v, out slices are then contiguous blocks of the caller's tensors in either layout
([B,H,T,d] or [B,T,H,d]) and its states are a contiguous block of [B,H,d,d].  No exchange step:
a caller that wants the whole output on every rank gathers it afterwards.

This module holds no arithmetic of the method, only index bookkeeping.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple


def batch_bounds(B: int, world: int, rank: int) -> Tuple[int, int]:
    """[b0, b1) of `rank`: contiguous, in rank order, sizes differing by at most one.  A rank
    may get an empty range when world > B (replicas only make sense then)."""
    if B < 0 or world < 1 or not 0 <= rank < world:
        raise ValueError("bad partition (B=%d, world=%d, rank=%d)" % (B, world, rank))
    return B * rank // world, B * (rank + 1) // world


def shard_batch(tensors: Sequence, world: int, rank: int):
    """The rank's slice along dim 0 of every tensor (None stays None); views, no copies."""
    out = []
    for t in tensors:
        if t is None:
            out.append(None)
            continue
        b0, b1 = batch_bounds(t.shape[0], world, rank)
        out.append(t[b0:b1])
    return out


def assemble_batch(parts: Sequence, B: Optional[int] = None):
    """Concatenate per-rank results (in rank order) along dim 0; checks the total batch."""
    import torch
    parts = [p for p in parts if p is not None and p.shape[0] > 0]
    full = torch.cat(parts, dim=0)
    if B is not None and full.shape[0] != B:
        raise ValueError("assembled batch %d != %d" % (full.shape[0], B))
    return full
