"""Stand-in for the inference engine that produced the rollouts, for building benchmark inputs.

The workload recipe says the sampled ids are drawn from the policy, softmax(hidden W^T), and that the
rollout engine's log-probs equal the true ones plus noise.  In training those come from a separate
inference engine; here a plain torch evaluation in row blocks plays that engine.  It is input synthesis
only: nothing in the library's path calls it, and its results are never used as expected values.
"""
from __future__ import annotations

import torch


@torch.no_grad()
def sample_tokens(hidden: torch.Tensor, W: torch.Tensor, u: torch.Tensor, block: int = 2048):
    """Returns (ids int32 [T], engine_logp float32 [T]): one token per row drawn by inverse CDF with the
    uniforms `u`, and the engine's log-probability of that token."""
    T = hidden.shape[0]
    ids = torch.empty(T, dtype=torch.int64, device=hidden.device)
    logp = torch.empty(T, dtype=torch.float32, device=hidden.device)
    for a in range(0, T, block):
        b = min(T, a + block)
        s = (hidden[a:b] @ W.T).float()
        lse = torch.logsumexp(s, dim=1)
        cdf = torch.cumsum(torch.exp(s - lse[:, None]).double(), dim=1)
        tgt = (u[a:b].double() * cdf[:, -1])[:, None]
        idx = torch.searchsorted(cdf, tgt, right=True).squeeze(1).clamp_(max=W.shape[0] - 1)
        ids[a:b] = idx
        logp[a:b] = s.gather(1, idx[:, None]).squeeze(1) - lse
    return ids.to(torch.int32), logp


@torch.no_grad()
def engine_logp(hidden: torch.Tensor, W: torch.Tensor, ids: torch.Tensor, block: int = 2048):
    """The engine's log-probability of given ids."""
    T = hidden.shape[0]
    logp = torch.empty(T, dtype=torch.float32, device=hidden.device)
    for a in range(0, T, block):
        b = min(T, a + block)
        s = (hidden[a:b] @ W.T).float()
        logp[a:b] = s.gather(1, ids[a:b].long()[:, None]).squeeze(1) - torch.logsumexp(s, dim=1)
    return logp
