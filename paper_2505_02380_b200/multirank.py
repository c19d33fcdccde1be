"""Host-side helpers for running the decode on several GPUs of one node.

The path has no exchange step (Section 3: segments decode independently), so ranks never
trade data.  Two things remain: deciding which tensors a rank decodes when one model is
split over the ranks, and reducing a per-rank timing to the slowest rank's.  Both work on
any torch.distributed backend (NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def shard_tensors(chunk_counts: Sequence[int], world: int) -> List[List[int]]:
    """Split tensors over `world` ranks so that the ranks' chunk totals are as even as a
    greedy longest-first assignment makes them.  chunk_counts[i] = chunks of tensor i.
    -> per rank, the tensor indices it decodes (ascending).  Deterministic, so every rank
    computes the same answer without communicating."""
    if world < 1:
        raise ValueError("world must be >= 1")
    order = sorted(range(len(chunk_counts)), key=lambda i: (-int(chunk_counts[i]), i))
    loads = [0] * world
    parts: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (loads[k], k))
        parts[r].append(i)
        loads[r] += int(chunk_counts[i])
    return [sorted(p) for p in parts]


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """The largest `value` any rank holds (the job's time is its slowest rank's).  A no-op
    without an initialised process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """Sum of `value` over ranks (units processed by the whole job)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
