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


def dw_shard_rows(V: int, v_chunk: int, world_size: int, rank: int):
    """Rows of dW that `rank` owns after reduce_scatter_dw_slices: of every slice [a, b) the rank-th of
    world_size equal parts of floor((b - a) / world_size) rows; the few rows left over at a slice's end go to
    the last rank.  Returns a list of (begin, end), one or two per slice, in row order."""
    out = []
    for a, b in chunk_slices(V, v_chunk):
        q = (b - a) // world_size
        if q > 0:
            out.append((a + rank * q, a + (rank + 1) * q))
        if rank == world_size - 1 and a + q * world_size < b:
            out.append((a + q * world_size, b))
    return out


def reduce_scatter_dw_slices(dW: torch.Tensor, v_chunk: int, shard: torch.Tensor, events=None, comm_stream=None):
    """Sums dW over the ranks slice by slice and leaves each rank with its rows only (what a trainer that shards
    the LM head's optimizer state needs: half the bytes of an all-reduce).

    `shard` [sum of owned rows, H] receives this rank's rows of the summed dW in the order of dw_shard_rows().
    Every slice is split into world_size equal parts (reduce-scatter); the fewer-than-world_size rows that may
    remain at its end are summed with a small all-reduce and kept by the last rank.  With `events` (one per slice,
    recorded by the library when the slice is final) the exchange of slice i runs on `comm_stream` while later
    slices are still being computed.  Returns the number of slices."""
    world = dist.get_world_size() if _multi() else 1
    rank = dist.get_rank() if _multi() else 0
    slices = chunk_slices(dW.shape[0], v_chunk)
    if events is not None:
        assert len(events) == len(slices)

    def exchange():
        pos = 0
        for i, (a, b) in enumerate(slices):
            if events is not None:
                comm_stream.wait_event(events[i])
            q = (b - a) // world
            if q > 0:
                dst = shard[pos:pos + q]
                if world > 1:
                    dist.reduce_scatter_tensor(dst, dW[a:a + q * world])
                else:
                    dst.copy_(dW[a:a + q])
                pos += q
            rest = (a + q * world, b)
            if rest[0] < rest[1]:
                if world > 1:
                    dist.all_reduce(dW[rest[0]:rest[1]])
                if rank == world - 1:
                    n = rest[1] - rest[0]
                    shard[pos:pos + n].copy_(dW[rest[0]:rest[1]])
                    pos += n
        return pos

    if events is None:
        pos = exchange()
    else:
        with torch.cuda.stream(comm_stream):
            pos = exchange()
    assert pos == shard.shape[0], "shard must hold exactly the rows of dw_shard_rows()"
    return len(slices)


# ---------------------------------------------------------------------------------------------
# Vocabulary-parallel LM head
# ---------------------------------------------------------------------------------------------

def vocab_shards(V: int, world_size: int, align: int = 256):
    """Contiguous row ranges [begin, end) of W, one per rank: equal multiples of `align` rows (the kernels'
    vocabulary tile), the last rank taking what is left.  Raises if some rank would get no rows at all (more
    ranks than vocabulary tiles): the library's calls need at least one row per range."""
    if V < 1 or world_size < 1:
        raise ValueError("vocab_shards: V and world_size must be positive")
    per = -(-V // world_size)
    per = -(-per // align) * align
    cuts = [(min(V, r * per), min(V, (r + 1) * per)) for r in range(world_size)]
    empty = [r for r, (a, b) in enumerate(cuts) if b <= a]
    if empty:
        raise ValueError(f"vocab_shards: {world_size} ranks over {V} rows in tiles of {align} leaves ranks {empty} "
                         "without rows; use fewer ranks or a smaller align")
    return cuts


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
    """Sums the ranks' parts of dH in place.  With more than one rank the parts must be fp32: a part rounded to
    bf16 before the sum loses bits that the sum of all parts would have kept."""
    if _multi():
        if dH_part.dtype not in (torch.float32, torch.float64):
            raise ValueError("all_reduce_dh: partial sums of dH cross the ranks in fp32 (set dh_dtype = DRK_F32 "
                             "and convert after the reduction)")
        dist.all_reduce(dH_part)
    return dH_part


def vocab_parallel_loss_fwd_bwd(hidden, W_shard, ids, rollout_logp, loss_mask, cu_seqlens, seg_adv, v_begin: int,
                                V_total: int, p, bufs, stats=None, stream=None, dh_out=None):
    """One fused loss step with W split by rows over the process group: statistics of this rank's rows,
    all-gather, loss and this rank's gradient parts, all-reduce of dH.  `bufs` is a PgLossBuffers built for
    V = W_shard.shape[0]; on return bufs.dW holds this rank's rows of dW and bufs.dH the complete dH.
    With more than one rank p.dh_dtype must be DRK_F32: every rank's dH is a partial sum, and the parts are added
    across the ranks in fp32 (dh_out, if given, receives the reduced dH converted to its own dtype)."""
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
    if dh_out is not None:
        dh_out.copy_(bufs.dH)
    return n_launch
