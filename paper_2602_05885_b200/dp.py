"""Multi-GPU plumbing around the library (which itself makes no collective call).

Data parallel: micro-batches are independent given the per-sample advantages, so ranks take disjoint
micro-batches and exchange nothing on the loss path; only timing is reduced, and dW by the trainer.
Vocabulary parallel: ranks hold row blocks of W, exchange per-row softmax statistics (all-gather of
16 bytes per token and rank) between the two library calls, and sum their parts of dH afterwards."""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist

from . import binding as B


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


# ---------------------------------------------------------------------------------------------
# Vocabulary-parallel LM head
# ---------------------------------------------------------------------------------------------

def vocab_shards(V: int, world_size: int, align: int = 256):
    """Contiguous row ranges [begin, end) of W, one per rank: equal multiples of `align` rows (the kernels'
    vocabulary tile), the last rank taking what is left.  Ranks beyond the vocabulary get empty ranges."""
    per = -(-V // world_size)
    per = -(-per // align) * align
    return [(min(V, r * per), min(V, (r + 1) * per)) for r in range(world_size)]


def _multi() -> bool:
    return dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1


def all_gather_stats(stats: torch.Tensor) -> torch.Tensor:
    """[T,4] per-rank statistics -> [world, T, 4], rank k's block at index k."""
    if not _multi():
        return stats.unsqueeze(0).contiguous()
    world = dist.get_world_size()
    out = torch.empty((world * stats.shape[0],) + tuple(stats.shape[1:]), dtype=stats.dtype, device=stats.device)
    dist.all_gather_into_tensor(out, stats.contiguous())      # concatenation along dim 0, in rank order
    return out.view((world,) + tuple(stats.shape))


def all_reduce_dh(dH_part: torch.Tensor) -> torch.Tensor:
    """Sums the ranks' parts of dH in place."""
    if _multi():
        dist.all_reduce(dH_part)
    return dH_part


def vocab_parallel_loss_fwd_bwd(hidden, W_shard, ids, rollout_logp, loss_mask, cu_seqlens, seg_adv, v_begin: int,
                                V_total: int, p, bufs, stats=None, stream=None):
    """One fused loss step with W split by rows over the process group: statistics of this rank's rows,
    all-gather, loss and this rank's gradient parts, all-reduce of dH.  `bufs` is a PgLossBuffers built for
    V = W_shard.shape[0]; on return bufs.dW holds this rank's rows of dW and bufs.dH the complete dH."""
    T, H = hidden.shape
    V_local = W_shard.shape[0]
    S = cu_seqlens.shape[0] - 1
    code = B.DRK_F32 if hidden.dtype == torch.float32 else B.DRK_BF16
    if stats is None:
        stats = torch.empty((T, 4), dtype=torch.float32, device=hidden.device)
    B.drk_pg_shard_stats_fwd(hidden, W_shard, code, ids, T, H, V_local, v_begin, V_total, p.engine, stats,
                             bufs.workspace, bufs.workspace_bytes, bufs.status, stream)
    n_launch = B.drk_last_launch_count()
    stats_all = all_gather_stats(stats)
    B.drk_pg_shard_loss_bwd(hidden, W_shard, code, ids, stats_all, stats_all.shape[0], rollout_logp, loss_mask,
                            cu_seqlens, seg_adv, T, H, V_local, v_begin, V_total, S, p, bufs.loss, bufs.logp, bufs.lse,
                            bufs.entropy, bufs.seg_w, bufs.seg_keep, bufs.counters, bufs.dH, bufs.dW, bufs.workspace,
                            bufs.workspace_bytes, bufs.status, stream)
    n_launch += B.drk_last_launch_count()
    all_reduce_dh(bufs.dH)
    return n_launch
