"""Seeded synthetic inputs shaped like multi-turn RL training batches.

This module only draws random numbers and lays out structure (group tables,
segment lengths, packing, masks).  It contains none of the method's arithmetic:
no returns, advantages, log-softmax, importance ratios or losses.  Quantities
that the workload recipe defines through the policy itself (token ids sampled
from softmax(hidden W^T); rollout log-probs = true log-probs + noise) are left
to the caller, who gets the raw uniforms `u_ids` and the additive `noise` and
combines them with log-probs from whichever implementation it is exercising.

Everything is a torch tensor; `device` may be "cpu" or a CUDA device.  A given
(seed, device type) always yields the same values.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


# ---------------------------------------------------------------------------
# Rollout batch: rewards, validity, group structure, response lengths
# ---------------------------------------------------------------------------

@dataclass
class RolloutBatch:
    P: int
    K: int
    Tmax: int
    reward: torch.Tensor             # [R, Tmax] float32
    valid: torch.Tensor              # [R, Tmax] uint8
    prompt_of_rollout: torch.Tensor  # [R] int32, non-decreasing
    resp_len: torch.Tensor           # [R, Tmax] int32 (0 where invalid)
    ctx_len: torch.Tensor            # [R, Tmax] int32 unmasked context tokens packed in front

    @property
    def R(self) -> int:
        return self.P * self.K


def draw_rewards(shape, gen: torch.Generator) -> torch.Tensor:
    """30 % exactly zero, otherwise U[0,1] + 0.5 * Bernoulli(0.3)."""
    zero = torch.rand(shape, generator=gen) < 0.3
    base = torch.rand(shape, generator=gen)
    bonus = (torch.rand(shape, generator=gen) < 0.3).float() * 0.5
    r = base + bonus
    r[zero] = 0.0
    return r.float()


def rollout_batch(P: int, K: int, Tmax: int, len_lo: int, len_hi: int, seed: int,
                  ragged: bool = False, ctx_frac: float = 0.0,
                  max_rollout_tokens: Optional[int] = None) -> RolloutBatch:
    """P prompts x K rollouts x up to Tmax turns.

    ragged=False: every rollout is valid at every turn.
    ragged=True : rollout i ends after turn tau_i ~ U{1..Tmax}; in addition the
    first prompt keeps a single rollout alive at the last turn (a group of
    one), the second prompt's rollouts all run to the end with equal rewards,
    and the third prompt's rewards are all zero (where those prompts exist).
    ctx_frac: fraction of each training sample that is unmasked context
    (prompt / feedback tokens) packed in front of the response.
    """
    g = _gen(seed, "cpu")
    R = P * K
    reward = draw_rewards((R, Tmax), g)
    valid = torch.ones((R, Tmax), dtype=torch.uint8)
    if ragged:
        tau = torch.randint(1, Tmax + 1, (R,), generator=g)
        turns = torch.arange(Tmax)[None, :]
        valid = (turns < tau[:, None]).to(torch.uint8)
        # a group of size one at the last turn of prompt 0
        valid[0:K, Tmax - 1] = 0
        valid[0, :] = 1
        if P > 1:   # all-equal, non-zero rewards on rollouts that all run to the last turn
            valid[K:2 * K, :] = 1
            reward[K:2 * K, :] = 1.25
        if P > 2:   # all-zero rewards
            reward[2 * K:3 * K, :] = 0.0
    reward = reward * valid.float()
    resp_len = torch.randint(len_lo, len_hi + 1, (R, Tmax), generator=g).to(torch.int32)
    resp_len = resp_len * valid.to(torch.int32)
    if ctx_frac > 0.0:
        ctx_len = (resp_len.float() * (ctx_frac / (1.0 - ctx_frac))).round().to(torch.int32)
    else:
        ctx_len = torch.zeros_like(resp_len)
    if max_rollout_tokens is not None:
        # shrink a rollout's turns proportionally if it exceeds the cap
        tot = (resp_len + ctx_len).sum(dim=1)
        over = tot > max_rollout_tokens
        if bool(over.any()):
            f = (max_rollout_tokens / tot.clamp(min=1).float()).clamp(max=1.0)[:, None]
            resp_len = torch.where(over[:, None], (resp_len.float() * f).floor().to(torch.int32), resp_len)
            ctx_len = torch.where(over[:, None], (ctx_len.float() * f).floor().to(torch.int32), ctx_len)
            resp_len = torch.maximum(resp_len, valid.to(torch.int32))  # keep >=1 token where valid
    prompt_of_rollout = torch.arange(P, dtype=torch.int32).repeat_interleave(K)
    return RolloutBatch(P, K, Tmax, reward, valid, prompt_of_rollout, resp_len, ctx_len)


# ---------------------------------------------------------------------------
# Packing of training samples ((rollout, turn) segments) into micro-batches
# ---------------------------------------------------------------------------

@dataclass
class Segment:
    rollout: int
    turn: int
    ctx: int     # unmasked tokens in front
    resp: int    # loss-masked response tokens

    @property
    def length(self) -> int:
        return self.ctx + self.resp


@dataclass
class MicroBatchPlan:
    T: int                       # packed tokens including tail padding
    segments: List[Segment] = field(default_factory=list)

    @property
    def used(self) -> int:
        return sum(s.length for s in self.segments)


def pack_first_fit(rb: RolloutBatch, capacity: int, pad_to_capacity: bool = True) -> List[MicroBatchPlan]:
    """First-fit packing of whole segments, in (rollout, turn) order, into
    micro-batches of at most `capacity` tokens.  A segment longer than the
    capacity is truncated to it (keeping the response tail)."""
    plans: List[MicroBatchPlan] = []
    for i in range(rb.R):
        for t in range(rb.Tmax):
            if not int(rb.valid[i, t]):
                continue
            seg = Segment(i, t, int(rb.ctx_len[i, t]), int(rb.resp_len[i, t]))
            if seg.length > capacity:
                seg.resp = min(seg.resp, capacity)
                seg.ctx = capacity - seg.resp
            for p in plans:
                if p.used + seg.length <= capacity:
                    p.segments.append(seg)
                    break
            else:
                plans.append(MicroBatchPlan(capacity, [seg]))
    if not pad_to_capacity:
        for p in plans:
            p.T = p.used
    return plans


def equal_segments_plan(T: int, K: int, Tmax: int) -> MicroBatchPlan:
    """Equal-length segments filling exactly T tokens (the sweep workload):
    as many (rollout, turn) samples of one common length as K*Tmax divides."""
    S = max(K * Tmax, 1)
    while S > 1 and T // S < 1:
        S -= 1
    base = T // S
    segs = []
    for j in range(S):
        ln = base + (T - base * S if j == S - 1 else 0)
        segs.append(Segment(j // Tmax, j % Tmax, 0, ln))
    return MicroBatchPlan(T, segs)


def plan_tensors(plan: MicroBatchPlan, lead_pad: int = 0):
    """cu_seqlens [S+1] int32, loss_mask [T] uint8, and the (rollout, turn)
    of every segment.  Tokens after the last segment are padding that belongs
    to no segment (`lead_pad` puts some in front as well)."""
    S = len(plan.segments)
    cu = torch.zeros(S + 1, dtype=torch.int32)
    mask = torch.zeros(plan.T, dtype=torch.uint8)
    pos = lead_pad
    cu[0] = pos
    for j, s in enumerate(plan.segments):
        mask[pos + s.ctx: pos + s.ctx + s.resp] = 1
        pos += s.length
        cu[j + 1] = pos
    assert pos <= plan.T
    seg_rollout = torch.tensor([s.rollout for s in plan.segments], dtype=torch.int64)
    seg_turn = torch.tensor([s.turn for s in plan.segments], dtype=torch.int64)
    return cu, mask, seg_rollout, seg_turn


# ---------------------------------------------------------------------------
# Dense operands and per-token random draws
# ---------------------------------------------------------------------------

def dense_operands(T: int, H: int, V: int, dtype: torch.dtype, seed: int, device="cpu",
                   distinct_rows: Optional[int] = None):
    """hidden ~ N(0,1) [T,H], W ~ N(0, 0.02^2) [V,H], rounded to `dtype`.

    distinct_rows=r draws only r different hidden rows and repeats them in a
    random order (row_of[t] tells which); the operands keep their full shape.
    """
    g = _gen(seed, device)
    W = torch.empty((V, H), dtype=torch.float32, device=device)
    # fill in slabs to bound temporary memory at large V*H
    step = max(1, (1 << 26) // H)
    for v0 in range(0, V, step):
        v1 = min(V, v0 + step)
        W[v0:v1].normal_(0.0, 0.02, generator=g)
    W = W.to(dtype)
    row_of = None
    if distinct_rows is None:
        hidden = torch.empty((T, H), dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g).to(dtype)
    else:
        base = torch.empty((distinct_rows, H), dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g).to(dtype)
        row_of = torch.randint(0, distinct_rows, (T,), generator=g, device=device)
        hidden = base[row_of].contiguous()
    return hidden, W, row_of


def token_draws(T: int, seed: int, device="cpu", sigma: float = 0.05,
                outlier_frac: float = 0.0, outlier_segments: Optional[torch.Tensor] = None,
                cu_seqlens: Optional[torch.Tensor] = None):
    """u_ids ~ U[0,1) for inverse-CDF sampling of token ids and the additive
    log-prob mismatch noise ~ N(0, sigma^2).

    outlier_frac > 0 overwrites that fraction of all tokens, chosen inside the
    segments flagged in `outlier_segments` only, with values of magnitude
    U[2,12] and random sign.
    """
    g = _gen(seed, device)
    u = torch.rand(T, generator=g, device=device, dtype=torch.float64)
    noise = torch.empty(T, dtype=torch.float32, device=device).normal_(0.0, sigma, generator=g)
    if outlier_frac > 0.0 and outlier_segments is not None and cu_seqlens is not None:
        inside = torch.zeros(T, dtype=torch.bool, device=device)
        cu = cu_seqlens.tolist()
        for j in outlier_segments.tolist():
            inside[cu[j]:cu[j + 1]] = True
        n_in = int(inside.sum())
        if n_in > 0:
            p = min(1.0, outlier_frac * T / n_in)
            pick = inside & (torch.rand(T, generator=g, device=device) < p)
            mag = 2.0 + 10.0 * torch.rand(T, generator=g, device=device)
            sign = torch.where(torch.rand(T, generator=g, device=device) < 0.5, -1.0, 1.0)
            noise = torch.where(pick, (mag * sign).float(), noise)
    return u, noise


def uniform_ids(T: int, V: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    return torch.randint(0, V, (T,), generator=g, device=device, dtype=torch.int64).to(torch.int32)


def pick_outlier_segments(S: int, frac: float, seed: int) -> torch.Tensor:
    g = _gen(seed, "cpu")
    n = max(1, int(round(S * frac))) if S > 0 else 0
    return torch.randperm(S, generator=g)[:n]


def threshold_between(values, spread: int = 2) -> float:
    """A threshold that splits `values` about in half without sitting on any of them: the midpoint of the
    widest gap between adjacent order statistics among the `spread` gaps either side of the median (fewer
    for short lists: one gap per eight values)."""
    a = sorted(float(v) for v in values)
    n = len(a)
    if n == 0:
        return 1e-3
    if n == 1:
        return 2.0 * a[0] if a[0] > 0 else 1e-3
    mid = n // 2
    spread = min(spread, n // 8)
    ks = range(max(0, mid - 1 - spread), min(n - 2, mid - 1 + spread) + 1)
    k = max(ks, key=lambda i: (a[i + 1] - a[i], -abs(i - (mid - 1))))
    return 0.5 * (a[k] + a[k + 1])
