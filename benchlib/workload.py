"""Named synthetic workloads (shapes and structure of the 8B / 14B multi-turn RL training batches)."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional

import torch

from . import rollout_sim, synth

CONFIGS = {
    # name: dtype, H, V, P, K, Tmax, len_lo, len_hi, capacity, sigma, outlier_frac, ragged, ctx_frac, ids
    "tiny": dict(dtype=torch.float32, H=256, V=4096, P=2, K=4, Tmax=2, len_lo=64, len_hi=64, capacity=1024,
                 sigma=0.05, outlier_frac=0.0, ragged=False, ctx_frac=0.0, ids="policy"),
    "qwen3-8b": dict(dtype=torch.bfloat16, H=4096, V=151936, P=16, K=8, Tmax=3, len_lo=128, len_hi=1024,
                     capacity=16384, sigma=0.05, outlier_frac=0.0, ragged=False, ctx_frac=0.0, ids="policy"),
    "qwen3-14b": dict(dtype=torch.bfloat16, H=5120, V=151936, P=32, K=8, Tmax=3, len_lo=256, len_hi=2048,
                      capacity=32768, sigma=0.1, outlier_frac=0.01, ragged=False, ctx_frac=0.0, ids="policy"),
    "ragged": dict(dtype=torch.bfloat16, H=5120, V=151936, P=32, K=8, Tmax=4, len_lo=128, len_hi=1228,
                   capacity=32768, sigma=0.1, outlier_frac=0.01, ragged=True, ctx_frac=0.4, ids="policy",
                   max_rollout_tokens=8192),
}


@dataclass
class Workload:
    name: str
    T: int
    H: int
    V: int
    S: int
    dtype: torch.dtype
    hidden: torch.Tensor
    W: torch.Tensor
    ids: torch.Tensor
    rollout_logp: torch.Tensor
    loss_mask: torch.Tensor
    cu: torch.Tensor
    seg_rollout: torch.Tensor
    seg_turn: torch.Tensor
    reward: torch.Tensor
    valid: torch.Tensor
    prompt_of_rollout: torch.Tensor
    noise: torch.Tensor
    row_of: Optional[torch.Tensor] = None
    n_microbatches: int = 1

    def wide_band(self):
        """(lo, hi) = exp(-+q) with q between two adjacent order statistics of the segments' |mean noise| next
        to their median: about half the samples pass, and no sample's mean lies on a threshold."""
        cu = self.cu.tolist()
        m = self.loss_mask.bool()
        vals = []
        for j in range(self.S):
            sel = m[cu[j]:cu[j + 1]]
            if int(sel.sum()) > 0:
                vals.append(abs(float(self.noise[cu[j]:cu[j + 1]][sel].mean())))
        q = synth.threshold_between(vals)
        return math.exp(-q), math.exp(q)


def build(name: str, device, seed: int = 2000, microbatch: int = 0, T_override: Optional[int] = None,
          distinct_rows: Optional[int] = None, sweep_shape=None) -> Workload:
    """Builds one packed micro-batch of the named config on `device`.

    sweep_shape=(T, V, H) gives a point of the roofline sweep instead: equal-length segments, uniform ids.
    """
    if sweep_shape is not None:
        T, V, H = sweep_shape
        c = dict(dtype=torch.bfloat16, H=H, V=V, P=1, K=8, Tmax=3, sigma=0.05, outlier_frac=0.0, ids="uniform")
        rb = synth.rollout_batch(1, 8, 3, 1, 1, seed)
        plan = synth.equal_segments_plan(T, 8, 3)
        n_mb = 1
    else:
        c = CONFIGS[name]
        rb = synth.rollout_batch(c["P"], c["K"], c["Tmax"], c["len_lo"], c["len_hi"], seed, ragged=c["ragged"],
                                 ctx_frac=c["ctx_frac"], max_rollout_tokens=c.get("max_rollout_tokens"))
        cap = T_override or c["capacity"]
        plans = synth.pack_first_fit(rb, cap)
        n_mb = len(plans)
        plan = plans[microbatch % n_mb]
        T, H, V = cap, c["H"], c["V"]
    cu, mask, seg_rollout, seg_turn = synth.plan_tensors(plan)
    S = cu.shape[0] - 1
    hidden, W, row_of = synth.dense_operands(T, H, V, c["dtype"], seed + 1, device, distinct_rows=distinct_rows)
    outl = synth.pick_outlier_segments(S, 0.1, seed + 3) if c["outlier_frac"] > 0 else None
    u, noise = synth.token_draws(T, seed + 2, device, sigma=c["sigma"], outlier_frac=c["outlier_frac"],
                                 outlier_segments=outl, cu_seqlens=cu)
    if c["ids"] == "uniform":
        ids = synth.uniform_ids(T, V, seed + 4, device)
        lp = rollout_sim.engine_logp(hidden, W, ids)
    else:
        ids, lp = rollout_sim.sample_tokens(hidden, W, u)
    rollout_logp = (lp + noise).float().contiguous()
    dev = torch.device(device)
    return Workload(name, T, H, V, S, c["dtype"], hidden, W, ids, rollout_logp, mask.to(dev), cu.to(dev),
                    seg_rollout.to(dev), seg_turn.to(dev), rb.reward.to(dev), rb.valid.to(dev),
                    rb.prompt_of_rollout.to(dev), noise, row_of, n_mb)
