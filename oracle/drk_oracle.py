"""fp64 CPU oracle for the fused policy-gradient loss over the LM head.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  Only the test-suite, the smoke check and the
CPU-baseline leg of the benchmark may import it; the product path never does.
It shares no code with the CUDA sources and never receives values produced by
them (the one exception is the documented `keep_override`, used by the parity
comparator for segments whose accept/reject decision lies inside rounding
distance of a threshold).

Everything is numpy float64.  `np.matmul` serves as the library primitive for
the three dense contractions; there is no blocking, fusion or reordering.

What follows the paper, and where:

  returns()            reward-to-go return                      Sec. 4.2, Eq. 2
  grpo_advantage()     turn-group mean baseline                 Sec. 4.2, Eq. 3
  trloo_advantage()    leave-one-out turn-level advantage       Sec. 4.2, Eq. 5
  mrs()                geometric mismatch rejection sampling    Sec. 5.1 (unnumbered eq.)
                       with the token-level veto
  coeff_and_loss()     REINFORCE surrogate                      App. A (estimator g-hat)
  segment_advantages()  advantage of the (rollout, turn) sample    Sec. 4.3 (every turn of a trajectory
                       a packed segment holds                   is one training sample)
  shard_stats()/merge_shard_stats()/shard_gradients()
                       the same definitions restricted to a range of vocabulary columns, and the
                       exact recombination of such ranges (the paper has no counterpart: this is
                       what each GPU of a vocabulary-split LM head can know on its own)
  logits()/token_logprob()/gradients()
                       the plain definition of log-softmax over the LM head
                       and its analytic gradient (the paper names the trainer
                       log-probability pi_train(a_t|s_t) but not how it is
                       computed; the definition is the textbook one).

Parity pins: every function here is pinned by tests that run without a GPU
(closed forms, brute force, finite differences, a float64 library
cross-check and the worked three-turn example of App. E); none is unpinned.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

F64 = np.float64

# Constants printed in Sec. 5.1.
MRS_LO = 0.999
MRS_HI = 1.001
MRS_VETO = 1e-4

NORM_KEPT_TOKENS = 0
NORM_ALL_MASKED_TOKENS = 1
NORM_EXPLICIT = 2


# ---------------------------------------------------------------------------
# Returns and advantages (Sec. 4.2)
# ---------------------------------------------------------------------------

def returns(reward, valid, gamma=1.0):
    """Eq. 2: G[i,t] = sum_{t'>=t} gamma^(t'-t) R[i,t'].

    A rollout that ended early has no reward at its later turns: only valid
    turns t' contribute, and an invalid (i,t) has G = 0.
    """
    reward = np.asarray(reward, dtype=F64)
    valid = np.asarray(valid).astype(bool)
    R, Tmax = reward.shape
    G = np.zeros((R, Tmax), dtype=F64)
    for i in range(R):
        for t in range(Tmax):
            if not valid[i, t]:
                continue
            acc = 0.0
            for tp in range(t, Tmax):
                if valid[i, tp]:
                    acc += (float(gamma) ** (tp - t)) * reward[i, tp]
            G[i, t] = acc
    return G


def turn_groups(valid, prompt_of_rollout):
    """The sets G_t of Sec. 4.2: for every prompt p and turn t, the valid
    rollouts of p at t.  Returns a list of (t, [rollout indices])."""
    valid = np.asarray(valid).astype(bool)
    prompt_of_rollout = np.asarray(prompt_of_rollout)
    R, Tmax = valid.shape
    groups = []
    for p in np.unique(prompt_of_rollout):
        members = [i for i in range(R) if prompt_of_rollout[i] == p]
        for t in range(Tmax):
            g = [i for i in members if valid[i, t]]
            if g:
                groups.append((t, g))
    return groups


def grpo_advantage(G, valid, prompt_of_rollout):
    """Eq. 3: A[i,t] = G[i,t] - mean_{j in G_t} G[j,t].  Returns (A, N)."""
    G = np.asarray(G, dtype=F64)
    A = np.zeros_like(G)
    N = np.zeros(G.shape, dtype=np.int64)
    for t, g in turn_groups(valid, prompt_of_rollout):
        n = len(g)
        mean = sum(G[j, t] for j in g) / n
        for i in g:
            A[i, t] = G[i, t] - mean
            N[i, t] = n
    return A, N


def trloo_advantage(G, valid, prompt_of_rollout):
    """Eq. 5: A[i,t] = G[i,t] - (1/(N_t-1)) sum_{j in G_t, j != i} G[j,t].

    The paper defines it for N_t > 1 only; a group of one has no other
    rollout to form a baseline from and gets advantage 0, as does every
    invalid (i,t).  Returns (A, N) with N[i,t] = N_t (0 where invalid).
    """
    G = np.asarray(G, dtype=F64)
    A = np.zeros_like(G)
    N = np.zeros(G.shape, dtype=np.int64)
    for t, g in turn_groups(valid, prompt_of_rollout):
        n = len(g)
        for i in g:
            N[i, t] = n
            if n > 1:
                others = sum(G[j, t] for j in g if j != i)
                A[i, t] = G[i, t] - others / (n - 1)
    return A, N


def segment_advantages(A, seg_rollout, seg_turn):
    """Sec. 4.3: each turn of a trajectory is one training sample.  Segment g of a packed micro-batch
    holds turn seg_turn[g] of rollout seg_rollout[g]; every token of it carries A[seg_rollout[g], seg_turn[g]]."""
    A = np.asarray(A, dtype=F64)
    out = np.zeros(len(seg_rollout), dtype=F64)
    for g in range(len(seg_rollout)):
        out[g] = A[int(seg_rollout[g]), int(seg_turn[g])]
    return out


# ---------------------------------------------------------------------------
# LM head: logits, log-softmax, gather
# ---------------------------------------------------------------------------

def logits(hidden, W):
    """s[t,v] = sum_h hidden[t,h] * W[v,h] (all of them)."""
    return np.matmul(np.asarray(hidden, dtype=F64), np.asarray(W, dtype=F64).T)


def logsumexp_rows(s):
    """lse[t] = max_v s[t,v] + ln sum_v exp(s[t,v] - max_v s[t,v])."""
    m = np.max(s, axis=1)
    return m + np.log(np.sum(np.exp(s - m[:, None]), axis=1))


def token_logprob(s, ids):
    """log pi(ids[t] | row t) = s[t, ids[t]] - lse[t].  Returns (logp, lse)."""
    ids = np.asarray(ids, dtype=np.int64)
    lse = logsumexp_rows(s)
    tgt = s[np.arange(s.shape[0]), ids]
    return tgt - lse, lse


# ---------------------------------------------------------------------------
# Mismatch rejection sampling (Sec. 5.1)
# ---------------------------------------------------------------------------

@dataclass
class MrsResult:
    w: np.ndarray           # [S] geometric-mean importance ratio
    keep: np.ndarray        # [S] bool
    vetoed: np.ndarray      # [S] bool, token veto fired
    mean_delta: np.ndarray  # [S] mean log ratio over the segment's masked tokens
    min_delta: np.ndarray   # [S] smallest token log ratio (+inf for empty segments)
    n_masked: np.ndarray    # [S] int64
    margin: np.ndarray      # [S] distance (log space) of the decision to the nearest threshold


def mrs(logp, rollout_logp, loss_mask, cu_seqlens, lo=MRS_LO, hi=MRS_HI, veto=MRS_VETO):
    """Geometric MRS with token veto, one decision per training sample.

    For the masked tokens M of a segment: delta_t = logp_t - rollout_logp_t,
    w = exp(mean_M delta).  The sample is retained iff lo <= w <= hi and no
    token's ratio exp(delta_t) is below `veto`.  Both tests are taken in log
    space (ln lo <= mean delta <= ln hi; min delta >= ln veto).  lo <= 0
    removes the lower bound, hi = inf the upper one, veto <= 0 the veto.
    A segment without masked tokens has w = 1 and is not retained.
    """
    logp = np.asarray(logp, dtype=F64)
    rollout_logp = np.asarray(rollout_logp, dtype=F64)
    loss_mask = np.asarray(loss_mask).astype(bool)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    S = cu.shape[0] - 1
    ln_lo = math.log(lo) if lo > 0 else -math.inf
    ln_hi = math.log(hi) if math.isfinite(hi) else math.inf
    ln_veto = math.log(veto) if veto > 0 else -math.inf
    w = np.ones(S, dtype=F64)
    keep = np.zeros(S, dtype=bool)
    vetoed = np.zeros(S, dtype=bool)
    mean_delta = np.zeros(S, dtype=F64)
    min_delta = np.full(S, np.inf, dtype=F64)
    n_masked = np.zeros(S, dtype=np.int64)
    margin = np.full(S, np.inf, dtype=F64)
    for g in range(S):
        a, b = int(cu[g]), int(cu[g + 1])
        m = loss_mask[a:b]
        n = int(m.sum())
        n_masked[g] = n
        if n == 0:
            continue
        delta = (logp[a:b] - rollout_logp[a:b])[m]
        mean_delta[g] = delta.sum() / n
        min_delta[g] = delta.min()
        w[g] = math.exp(mean_delta[g])
        in_band = (ln_lo <= mean_delta[g]) and (mean_delta[g] <= ln_hi)
        vetoed[g] = min_delta[g] < ln_veto
        keep[g] = in_band and not vetoed[g]
        margin[g] = min(abs(mean_delta[g] - ln_lo), abs(mean_delta[g] - ln_hi),
                        abs(min_delta[g] - ln_veto))
    return MrsResult(w, keep, vetoed, mean_delta, min_delta, n_masked, margin)


# ---------------------------------------------------------------------------
# Coefficients and the loss (App. A)
# ---------------------------------------------------------------------------

@dataclass
class LossResult:
    coeff: np.ndarray     # [T] coefficient c_t that multiplies grad log pi at token t
    loss: float
    scale: float
    kept_tokens: int
    masked_tokens: int
    kept_segs: int


def coeff_and_loss(logp, keep, loss_mask, cu_seqlens, seg_adv,
                   norm=NORM_KEPT_TOKENS, explicit_scale=1.0):
    """c_t = keep_seg(t) * mask_t * A_seg(t) * scale, loss = -sum_t c_t logp_t.

    The estimator of App. A sums grad log pi(y_{i,t}|s_{i,t}) * A_{i,t} over
    samples; log pi of a response is the sum of its token log-probs, so every
    masked token of a retained sample carries the sample's advantage.  The
    outer averaging convention is left open by the paper: `norm` picks
    1/(kept masked tokens), 1/(all masked tokens) or a caller constant.
    Tokens outside [cu[0], cu[S]) belong to no sample and get c_t = 0.
    """
    logp = np.asarray(logp, dtype=F64)
    loss_mask = np.asarray(loss_mask).astype(bool)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    keep = np.asarray(keep).astype(bool)
    seg_adv = np.asarray(seg_adv, dtype=F64)
    S = cu.shape[0] - 1
    T = logp.shape[0]
    kept_tokens = 0
    masked_tokens = 0
    for g in range(S):
        n = int(loss_mask[cu[g]:cu[g + 1]].sum())
        masked_tokens += n
        if keep[g]:
            kept_tokens += n
    if norm == NORM_KEPT_TOKENS:
        scale = 1.0 / max(kept_tokens, 1)
    elif norm == NORM_ALL_MASKED_TOKENS:
        scale = 1.0 / max(masked_tokens, 1)
    elif norm == NORM_EXPLICIT:
        scale = float(explicit_scale)
    else:
        raise ValueError("unknown norm")
    coeff = np.zeros(T, dtype=F64)
    for g in range(S):
        if not keep[g]:
            continue
        a, b = int(cu[g]), int(cu[g + 1])
        coeff[a:b] = np.where(loss_mask[a:b], seg_adv[g] * scale, 0.0)
    loss = -float(np.sum(coeff * logp))
    return LossResult(coeff, loss, scale, kept_tokens, masked_tokens, int(keep.sum()))


# ---------------------------------------------------------------------------
# Gradients of the loss w.r.t. hidden and W (c_t held constant)
# ---------------------------------------------------------------------------

def dlogits(s, lse, ids, coeff):
    """dL[t,v] = c_t * (softmax(s)[t,v] - [v == ids[t]])."""
    p = np.exp(s - np.asarray(lse, dtype=F64)[:, None])
    p[np.arange(s.shape[0]), np.asarray(ids, dtype=np.int64)] -= 1.0
    return p * np.asarray(coeff, dtype=F64)[:, None]


def gradients(hidden, W, s, lse, ids, coeff):
    """dH[t,:] = sum_v dL[t,v] W[v,:];  dW[v,:] = sum_t dL[t,v] hidden[t,:]."""
    dL = dlogits(s, lse, ids, coeff)
    dH = np.matmul(dL, np.asarray(W, dtype=F64))
    dW = np.matmul(dL.T, np.asarray(hidden, dtype=F64))
    return dH, dW


# ---------------------------------------------------------------------------
# The same quantities when the vocabulary is split into column ranges (one range per GPU)
# ---------------------------------------------------------------------------

def shard_stats(s, ids, v_begin, v_end):
    """What the owner of columns [v_begin, v_end) knows about each row t, from its own logits only:
    m = max_v s[t,v];  l = sum_v exp(s[t,v] - m);  r = sum_v exp(s[t,v] - m) * s[t,v];
    g = s[t, ids[t]] if v_begin <= ids[t] < v_end else 0.   Returns an array [T, 4] = (m, l, r, g)."""
    s = np.asarray(s, dtype=F64)
    ids = np.asarray(ids, dtype=np.int64)
    T = s.shape[0]
    out = np.zeros((T, 4), dtype=F64)
    for t in range(T):
        row = s[t, v_begin:v_end]
        m = row.max()
        e = np.exp(row - m)
        out[t, 0] = m
        out[t, 1] = e.sum()
        out[t, 2] = (e * row).sum()
        if v_begin <= ids[t] < v_end:
            out[t, 3] = s[t, ids[t]]
    return out


def merge_shard_stats(stats):
    """Recombines shard_stats of ranges that partition the vocabulary (stats: [n, T, 4]):
    M = max_k m_k;  L = sum_k l_k exp(m_k - M);  lse = M + ln L;  logp = sum_k g_k - lse;
    entropy = lse - (sum_k r_k exp(m_k - M)) / L.   Returns (logp, lse, entropy)."""
    st = np.asarray(stats, dtype=F64)
    M = st[:, :, 0].max(axis=0)
    wgt = np.exp(st[:, :, 0] - M[None, :])
    L = (st[:, :, 1] * wgt).sum(axis=0)
    Rr = (st[:, :, 2] * wgt).sum(axis=0)
    lse = M + np.log(L)
    return st[:, :, 3].sum(axis=0) - lse, lse, lse - Rr / L


def shard_gradients(hidden, W, s, lse, ids, coeff, v_begin, v_end):
    """The part of the gradients that the owner of columns [v_begin, v_end) forms from them alone:
    dH_part[t,:] = sum_{v in range} dL[t,v] W[v,:]  (the ranges' parts add up to dH);
    dW_rows[v,:] = sum_t dL[t,v] hidden[t,:] for v in the range (rows v_begin..v_end of dW)."""
    dL = dlogits(s, lse, ids, coeff)[:, v_begin:v_end]
    dH_part = np.matmul(dL, np.asarray(W, dtype=F64)[v_begin:v_end])
    dW_rows = np.matmul(dL.T, np.asarray(hidden, dtype=F64))
    return dH_part, dW_rows


# ---------------------------------------------------------------------------
# The whole path for one packed micro-batch
# ---------------------------------------------------------------------------

def pg_loss_fwd_bwd(hidden, W, ids, rollout_logp, loss_mask, cu_seqlens, seg_adv,
                    lo=MRS_LO, hi=MRS_HI, veto=MRS_VETO,
                    norm=NORM_KEPT_TOKENS, explicit_scale=1.0,
                    keep_override=None, want_grads=True):
    """Forward, MRS, loss and (optionally) gradients.  Returns a dict."""
    s = logits(hidden, W)
    logp, lse = token_logprob(s, ids)
    m = mrs(logp, rollout_logp, loss_mask, cu_seqlens, lo, hi, veto)
    keep = m.keep if keep_override is None else np.asarray(keep_override).astype(bool)
    lr = coeff_and_loss(logp, keep, loss_mask, cu_seqlens, seg_adv, norm, explicit_scale)
    out = dict(logp=logp, lse=lse, mrs=m, keep=keep, coeff=lr.coeff, loss=lr.loss,
               scale=lr.scale, kept_tokens=lr.kept_tokens, masked_tokens=lr.masked_tokens,
               kept_segs=lr.kept_segs, vetoed_segs=int(m.vetoed.sum()))
    if want_grads:
        dH, dW = gradients(hidden, W, s, lse, ids, lr.coeff)
        out["dH"] = dH
        out["dW"] = dW
    return out


# ---------------------------------------------------------------------------
# Reward front-end (Sec. 4.2 Eq. 1; Sec. 5.2 profiling-based reward and rejection sampling)
# ---------------------------------------------------------------------------

def speedup_reward(correct, t_ref, t_kernel, pr=None, clip=3.0):
    """Eq. 1: R = C + C * min(T_ref / T_kernel, clip).  With a profiling ratio (Sec. 5.2) the
    reward of a correct kernel additionally gains PR = T_generated / T_total."""
    C = np.asarray(correct).astype(bool)
    speed = np.minimum(np.asarray(t_ref, dtype=F64) / np.asarray(t_kernel, dtype=F64), float(clip))
    R = np.where(C, 1.0 + speed, 0.0)
    if pr is not None:
        R = R + np.where(C, np.asarray(pr, dtype=F64), 0.0)
    return R


def prs_keep_prob(pr, tau=0.3, s=0.1):
    """Sec. 5.2: p = clip((PR - tau) / s, 0, 1).  Taken in float32 (subtract, divide, clamp), the
    precision in which the retention decision is made."""
    pr32 = np.asarray(pr, dtype=np.float32)
    p = (pr32 - np.float32(tau)) / np.float32(s)
    return np.minimum(np.maximum(p, np.float32(0.0)), np.float32(1.0)).astype(np.float32)


_PHILOX_M0, _PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
_PHILOX_W0, _PHILOX_W1 = 0x9E3779B9, 0xBB67AE85
_MASK32 = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as
    1, 2, 3", SC'11), written from its definition with Python integers."""
    c0, c1, c2, c3 = [int(x) & _MASK32 for x in counter]
    k0, k1 = [int(x) & _MASK32 for x in key]
    for r in range(10):
        if r > 0:
            k0 = (k0 + _PHILOX_W0) & _MASK32
            k1 = (k1 + _PHILOX_W1) & _MASK32
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK32
        hi1, lo1 = p1 >> 32, p1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK32, lo1, (hi0 ^ c3 ^ k1) & _MASK32, lo0
    return c0, c1, c2, c3


def prs_uniform(seed, offset, index):
    """The uniform in [0,1) that decides sample `index`: the top 24 bits of the first output word
    of Philox-4x32-10 with key = seed (low, high word) and counter = (index, offset) (low, high
    words each), scaled by 2^-24 (exact in float32)."""
    x0 = philox4x32_10((index & _MASK32, (index >> 32) & _MASK32, offset & _MASK32, (offset >> 32) & _MASK32),
                       (seed & _MASK32, (seed >> 32) & _MASK32))[0]
    return np.float32((x0 >> 8) * (1.0 / 16777216.0))


PRS_OFF, PRS_SOFT, PRS_HARD = 0, 1, 2


def prs_retain(pr, tau=0.3, s=0.1, mode=PRS_SOFT, seed=0, offset=0):
    """Profiling-based rejection sampling: sample i is retained with probability p_i (soft), or iff
    PR_i >= tau (the hard-threshold variant of the PRS ablation, App. D), or always (off)."""
    pr = np.asarray(pr, dtype=np.float32)
    n = pr.shape[0]
    if mode == PRS_OFF:
        return np.ones(n, dtype=bool)
    if mode == PRS_HARD:
        return pr >= np.float32(tau)
    p = prs_keep_prob(pr, tau, s)
    u = np.array([prs_uniform(seed, offset, i) for i in range(n)], dtype=np.float32)
    return u < p


# ---------------------------------------------------------------------------
# Stability diagnostics (the quantities monitored in Sec. 5.1 / App. B: entropy, perplexities of the
# trainer and of the rollout engine, log-ratio statistics, gradient norms)
# ---------------------------------------------------------------------------

def token_entropy(s):
    """Entropy of softmax(s[t,:]) per row: H_t = -sum_v p_v ln p_v = lse_t - sum_v p_v s_v."""
    lse = logsumexp_rows(s)
    p = np.exp(s - lse[:, None])
    return lse - np.sum(p * s, axis=1)


def diagnostics(logp, rollout_logp, entropy, loss_mask, cu_seqlens, dH=None, dW=None):
    """Means over the loss-masked tokens that lie inside segments.  Returns a dict:
    n_tokens, mean_entropy, ppl_train = exp(-mean logp), ppl_rollout = exp(-mean rollout_logp),
    mean_log_ratio = mean(logp - rollout_logp), max_abs_log_ratio, grad_norm_dH, grad_norm_dW
    (Frobenius norms; 0 when the gradient is not given)."""
    logp = np.asarray(logp, dtype=F64)
    rl = np.asarray(rollout_logp, dtype=F64)
    mask = np.asarray(loss_mask).astype(bool)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    sel = np.zeros(logp.shape[0], dtype=bool)
    for g in range(cu.shape[0] - 1):
        sel[cu[g]:cu[g + 1]] = True
    sel &= mask
    n = int(sel.sum())
    out = dict(n_tokens=n, mean_entropy=0.0, ppl_train=1.0, ppl_rollout=1.0, mean_log_ratio=0.0,
               max_abs_log_ratio=0.0, grad_norm_dH=0.0, grad_norm_dW=0.0)
    if n > 0:
        d = logp[sel] - rl[sel]
        out["mean_entropy"] = float(np.asarray(entropy, dtype=F64)[sel].sum() / n) if entropy is not None else 0.0
        out["ppl_train"] = math.exp(-float(logp[sel].sum()) / n)
        out["ppl_rollout"] = math.exp(-float(rl[sel].sum()) / n)
        out["mean_log_ratio"] = float(d.sum() / n)
        out["max_abs_log_ratio"] = float(np.abs(d).max())
    if dH is not None:
        out["grad_norm_dH"] = float(np.sqrt(np.sum(np.asarray(dH, dtype=F64) ** 2)))
    if dW is not None:
        out["grad_norm_dW"] = float(np.sqrt(np.sum(np.asarray(dW, dtype=F64) ** 2)))
    return out
