"""Data-parallel plumbing: micro-batches are independent given the per-sample advantages, so ranks
take disjoint micro-batches and exchange nothing on the loss path.  Only timing is reduced."""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def assign_microbatches(loads: Sequence[int], world_size: int) -> List[List[int]]:
    """Greedy longest-first assignment of micro-batches (by token count) to ranks; returns, per rank, the
    indices it owns.  Every micro-batch goes to exactly one rank."""
    order = sorted(range(len(loads)), key=lambda i: (-loads[i], i))
    owned: List[List[int]] = [[] for _ in range(world_size)]
    total = [0] * world_size
    for i in order:
        r = min(range(world_size), key=lambda k: (total[k], k))
        owned[r].append(i)
        total[r] += loads[i]
    return [sorted(o) for o in owned]


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` across the process group (the job's time is its slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
