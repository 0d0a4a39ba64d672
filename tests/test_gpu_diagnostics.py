"""drk_pg_diagnostics (and the entropy output of the forward kernels) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import drk_oracle as O
from paper_2602_05885_b200 import binding as B
from tests import helpers as Hh
from tests.gpu_utils import make_params

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,engine", [(torch.float32, B.DRK_ENGINE_AUTO), (torch.bfloat16, B.DRK_ENGINE_AUTO),
                                          (torch.bfloat16, B.DRK_ENGINE_UMMA_1CTA), (torch.bfloat16, B.DRK_ENGINE_SIMT)])
def test_diagnostics_after_a_loss_call(dtype, engine):
    d = torch.device("cuda:0")
    case = Hh.build_case("diag", H=256, V=4200, dtype=dtype, P=4, K=4, Tmax=2, len_lo=16, len_hi=64,
                         capacity=900, seed=31, sigma=0.1, outlier_frac=0.02, ctx_frac=0.3, lead_pad=3)
    p = make_params(0.0, float("inf"), 0.0, engine=engine, dh_dtype=B.DRK_BF16 if dtype == torch.bfloat16 else B.DRK_F32)
    code = B.DRK_F32 if dtype == torch.float32 else B.DRK_BF16
    bufs = B.PgLossBuffers(case.T, case.H, case.V, case.S, code, p, d)
    B.pg_loss_fwd_bwd(case.hidden.to(d), case.W.to(d), case.ids.to(d), case.rollout_logp.to(d), case.loss_mask.to(d),
                      case.cu.to(d), case.seg_adv.to(d), p, bufs)
    out = torch.empty(8, dtype=torch.float64, device=d)
    B.drk_pg_diagnostics(bufs.logp, case.rollout_logp.to(d), bufs.entropy, case.loss_mask.to(d), case.cu.to(d), case.T,
                         case.S, bufs.dH, p.dh_dtype, bufs.dW, p.dw_dtype, case.H, case.V, out)
    assert B.drk_last_launch_count() == 4
    torch.cuda.synchronize()
    got = dict(zip(B.DIAG_FIELDS, out.cpu().tolist()))
    tol = Hh.TOL_LOGP_F32 if dtype == torch.float32 else Hh.TOL_LOGP_BF16
    ent = O.token_entropy(case.s)
    assert np.abs(Hh.f64(bufs.entropy) - ent).max() <= tol
    ref_all = Hh.oracle_eval(case, 0.0, float("inf"), 0.0)
    ref = O.diagnostics(case.logp, Hh.f64(case.rollout_logp), ent, case.loss_mask.numpy(), case.cu.numpy(),
                        ref_all["dH"], ref_all["dW"])
    assert got["n_tokens"] == ref["n_tokens"] > 0
    assert abs(got["mean_entropy"] - ref["mean_entropy"]) <= tol
    assert abs(got["ppl_train"] / ref["ppl_train"] - 1) <= 2 * tol
    assert abs(got["ppl_rollout"] / ref["ppl_rollout"] - 1) <= 1e-6
    assert abs(got["mean_log_ratio"] - ref["mean_log_ratio"]) <= tol
    assert abs(got["max_abs_log_ratio"] - ref["max_abs_log_ratio"]) <= tol
    assert abs(got["grad_norm_dH"] / ref["grad_norm_dH"] - 1) <= Hh.TOL_GRAD_FRO
    assert abs(got["grad_norm_dW"] / ref["grad_norm_dW"] - 1) <= Hh.TOL_GRAD_FRO


def test_diagnostics_optional_inputs_and_empty():
    d = torch.device("cuda:0")
    T = 100
    logp = -torch.rand(T, device=d) * 3
    rl = logp - 0.25
    mask = torch.ones(T, dtype=torch.uint8, device=d)
    cu = torch.tensor([0, 40, 100], dtype=torch.int32, device=d)
    out = torch.full((8,), -1.0, dtype=torch.float64, device=d)
    B.drk_pg_diagnostics(logp, rl, None, mask, cu, T, 2, None, 0, None, 0, 8, 16, out)
    torch.cuda.synchronize()
    g = dict(zip(B.DIAG_FIELDS, out.cpu().tolist()))
    assert g["n_tokens"] == 100 and g["mean_entropy"] == 0 and g["grad_norm_dH"] == 0 and g["grad_norm_dW"] == 0
    assert abs(g["mean_log_ratio"] - 0.25) < 1e-6 and abs(g["max_abs_log_ratio"] - 0.25) < 1e-6
    assert abs(g["ppl_rollout"] / g["ppl_train"] - np.exp(0.25)) < 1e-5
    B.drk_pg_diagnostics(logp, rl, None, mask, cu, T, 0, None, 0, None, 0, 8, 16, out)     # no segments
    torch.cuda.synchronize()
    g = dict(zip(B.DIAG_FIELDS, out.cpu().tolist()))
    assert g["n_tokens"] == 0 and g["ppl_train"] == 1.0 and g["ppl_rollout"] == 1.0
