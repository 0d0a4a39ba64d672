"""Runs the CUDA path (through the C ABI binding) on a test case; no oracle code here."""
from __future__ import annotations

import torch

from paper_2602_05885_b200 import binding as B


def make_params(lo=None, hi=None, veto=None, norm=0, explicit_scale=1.0, dw_dtype=B.DRK_F32, dh_dtype=B.DRK_F32,
                dw_accumulate=0, engine=B.DRK_ENGINE_AUTO, v_chunk=0, keep_from_caller=0, forward_rows=0,
                reuse_forward=0, schedule=B.DRK_SCHEDULE_DYNAMIC):
    p = B.drk_pg_params_default()
    if lo is not None:
        p.mrs_lo = lo
    if hi is not None:
        p.mrs_hi = hi
    if veto is not None:
        p.veto_ratio = veto
    p.norm = norm
    p.explicit_scale = explicit_scale
    p.dw_dtype = dw_dtype
    p.dh_dtype = dh_dtype
    p.dw_accumulate = dw_accumulate
    p.engine = engine
    p.v_chunk = v_chunk
    p.keep_from_caller = keep_from_caller
    p.forward_rows = forward_rows
    p.reuse_forward = reuse_forward
    p.schedule = schedule
    return p


def run_device(case, p, seg_adv=None, dW_init=None, device="cuda:0", keep_in=None, logp_in=None, lse_in=None):
    dev = torch.device(device)
    hidden = case.hidden.to(dev)
    W = case.W.to(dev)
    ids = case.ids.to(dev)
    rl = case.rollout_logp.to(dev)
    mask = case.loss_mask.to(dev)
    cu = case.cu.to(dev)
    adv = (case.seg_adv if seg_adv is None else seg_adv).to(dev)
    code = B.DRK_F32 if case.dtype == torch.float32 else B.DRK_BF16
    dW = dW_init.to(dev).clone() if dW_init is not None else None
    bufs = B.PgLossBuffers(case.T, case.H, case.V, case.S, code, p, dev, dW=dW)
    # poison outputs so that unwritten elements show
    bufs.dH.fill_(float("nan"))
    if dW_init is None:
        bufs.dW.fill_(float("nan"))
    bufs.logp.fill_(float("nan"))
    if logp_in is not None:
        bufs.logp.copy_(logp_in.to(dev))
        bufs.lse.copy_(lse_in.to(dev))
    if keep_in is not None:
        bufs.seg_keep.copy_(keep_in.to(dev))
    B.pg_loss_fwd_bwd(hidden, W, ids, rl, mask, cu, adv, p, bufs)
    torch.cuda.synchronize()
    out = dict(logp=bufs.logp.cpu(), lse=bufs.lse.cpu(), entropy=bufs.entropy.cpu(), seg_w=bufs.seg_w.cpu(), seg_keep=bufs.seg_keep.cpu(),
               loss=bufs.loss.cpu(), counters=bufs.counters.cpu(), dH=bufs.dH.float().cpu(),
               dW=bufs.dW.float().cpu(), status=int(bufs.status.cpu().item()), launches=B.drk_last_launch_count())
    return out
