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


def chunk_slices(V: int, v_chunk: int):
    """Row ranges [a, b) of dW that the backward finishes one after the other."""
    return [(a, min(V, a + v_chunk)) for a in range(0, V, v_chunk)]


def all_reduce_dw_slices(dW: torch.Tensor, v_chunk: int, events=None, comm_stream=None):
    """Sums dW over the ranks slice by slice, in the order in which the backward finishes the slices.

    On a GPU, `events[i]` (recorded by the library when slice i is final) gates slice i on `comm_stream`,
    so the reduction of early slices overlaps the computation of later ones.  Without events (CPU tensors,
    gloo) the slices are reduced one after the other.  Returns the number of slices.
    """
    slices = chunk_slices(dW.shape[0], v_chunk)
    multi = dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1
    if events is None:
        for a, b in slices:
            if multi:
                dist.all_reduce(dW[a:b])
        return len(slices)
    assert len(events) == len(slices)
    with torch.cuda.stream(comm_stream):
        for (a, b), e in zip(slices, events):
            comm_stream.wait_event(e)
            if multi:
                dist.all_reduce(dW[a:b])
    return len(slices)
