"""Edge cases of the device path: ragged and degenerate sizes, bad inputs that only the device can see."""
import math

import numpy as np
import pytest
import torch

from paper_2602_05885_b200 import binding as B
from tests import helpers as Hh
from tests.gpu_utils import make_params, run_device

pytestmark = pytest.mark.gpu

OPEN = (0.0, math.inf, 0.0)      # MRS switched off: every sample with a masked token is retained


@pytest.mark.parametrize("T,H,V", [(1, 64, 300), (127, 264, 4104), (129, 72, 4099), (300, 512, 257), (64, 8, 1)])
@pytest.mark.parametrize("dtype,engine", [(torch.bfloat16, B.DRK_ENGINE_AUTO), (torch.bfloat16, B.DRK_ENGINE_UMMA_1CTA),
                                          (torch.float32, B.DRK_ENGINE_AUTO)])
def test_ragged_sizes(T, H, V, dtype, engine):
    case = Hh.build_plain_case(f"r{T}_{H}_{V}", T=T, H=H, V=V, dtype=dtype, S=3, seed=T + V, mask_frac=0.2)
    dev = run_device(case, make_params(*OPEN, v_chunk=256, engine=engine))
    assert dev["status"] == 0
    Hh.check_against_oracle(case, dev, *OPEN)


def test_all_rejected_gives_exact_zero():
    case = Hh.build_plain_case("rej", T=200, H=128, V=1000, dtype=torch.bfloat16, S=4, seed=11, sigma=0.5)
    lo, hi, veto = float(np.float32(0.999999)), float(np.float32(1.000001)), float(np.float32(1e-4))
    dev = run_device(case, make_params(lo, hi, veto))
    ref = Hh.check_against_oracle(case, dev, lo, hi, veto)
    assert ref["kept_segs"] == 0
    assert float(dev["loss"]) == 0.0 and (dev["dH"] == 0).all() and (dev["dW"] == 0).all()


def test_empty_inputs():
    d = torch.device("cuda:0")
    # S = 0: nothing to train on
    case = Hh.build_plain_case("s0", T=130, H=64, V=500, dtype=torch.bfloat16, S=1, seed=12)
    case.cu = torch.zeros(1, dtype=torch.int32)
    case.seg_adv = torch.zeros(0)
    dev = run_device(case, make_params(*OPEN))
    assert float(dev["loss"]) == 0.0 and (dev["dH"] == 0).all() and (dev["dW"] == 0).all()
    assert (dev["counters"] == 0).all()
    assert np.abs(Hh.f64(dev["logp"]) - case.logp).max() <= Hh.TOL_LOGP_BF16
    # T = 0
    H, V = 64, 512
    W = torch.randn(V, H).to(torch.bfloat16).to(d)
    p = make_params(*OPEN)
    bufs = B.PgLossBuffers(0, H, V, 2, B.DRK_BF16, p, d)
    bufs.dW.fill_(1.0)
    e = torch.empty(0, device=d)
    cu = torch.zeros(3, dtype=torch.int32, device=d)
    B.drk_pg_loss_fwd_bwd(e, W, B.DRK_BF16, e, e, e, cu, torch.ones(2, device=d), 0, H, V, 2, p, bufs.loss, bufs.logp,
                          bufs.lse, None, bufs.seg_w, bufs.seg_keep, bufs.counters, bufs.dH, bufs.dW, bufs.workspace,
                          bufs.workspace_bytes, bufs.status)
    torch.cuda.synchronize()
    assert float(bufs.loss.item()) == 0.0 and (bufs.dW == 0).all() and (bufs.seg_keep == 0).all()
    assert (bufs.seg_w == 1).all()
    assert B.drk_pg_logprob_fwd(e, W, B.DRK_BF16, e, 0, H, V, 0, e, e, None, bufs.workspace, bufs.workspace_bytes,
                                bufs.status) == B.DRK_OK


def test_device_detected_errors_set_status_bits():
    case = Hh.build_plain_case("bad", T=140, H=64, V=700, dtype=torch.bfloat16, S=2, seed=13)
    good = case.ids.clone()
    case.ids[5] = 700          # outside [0, V)
    case.ids[9] = -3
    dev = run_device(case, make_params(*OPEN))
    assert dev["status"] & B.DRK_STATUS_BAD_ID
    ok = np.ones(140, dtype=bool)
    ok[[5, 9]] = False
    assert np.abs(Hh.f64(dev["logp"]) - case.logp)[ok].max() <= Hh.TOL_LOGP_BF16
    # a bad row's target logit reads as 0, so logp = -lse
    assert abs(float(dev["logp"][5]) + float(dev["lse"][5])) < 1e-6
    case.ids = good
    case.cu = torch.tensor([0, 90, 60], dtype=torch.int32)      # decreasing
    dev = run_device(case, make_params(*OPEN))
    assert dev["status"] & B.DRK_STATUS_BAD_SEGMENTS
    assert int(dev["seg_keep"][1]) == 0
    # boundaries that go back and forward again would make two samples share tokens: the step back is what
    # the device sees, and it raises the same bit
    case.cu = torch.tensor([0, 90, 40, 140], dtype=torch.int32)
    case.seg_adv = torch.ones(3)
    dev = run_device(case, make_params(*OPEN))
    assert dev["status"] & B.DRK_STATUS_BAD_SEGMENTS
    assert int(dev["seg_keep"][1]) == 0


def test_host_detected_errors_return_codes():
    d = torch.device("cuda:0")
    T, H, V = 64, 64, 256
    hidden = torch.zeros((T, H), dtype=torch.bfloat16, device=d)
    W = torch.zeros((V, H), dtype=torch.bfloat16, device=d)
    ids = torch.zeros(T, dtype=torch.int32, device=d)
    logp = torch.empty(T, device=d)
    lse = torch.empty(T, device=d)
    st = torch.zeros(1, dtype=torch.int32, device=d)
    nb = B.drk_pg_workspace_bytes(T, H, V, 0, B.DRK_BF16, None, 0)
    ws = torch.empty(nb, dtype=torch.uint8, device=d)
    call = lambda **kw: B.drk_pg_logprob_fwd(kw.get("hidden", hidden), W, kw.get("dt", B.DRK_BF16), ids,
                                             kw.get("T", T), kw.get("H", H), V, 0, logp, lse, None, ws,
                                             kw.get("nb", nb), st, check=False)
    assert call() == B.DRK_OK
    assert call(nb=nb - 512) == B.DRK_ERR_WORKSPACE
    assert call(T=-1) == B.DRK_ERR_INVALID_ARG
    assert call(dt=7) == B.DRK_ERR_INVALID_ARG
    assert call(H=68) == B.DRK_ERR_UNSUPPORTED            # bf16 rows must be 16-byte multiples
    assert call(hidden=hidden.view(-1)[1:]) == B.DRK_ERR_INVALID_ARG   # misaligned
    assert B.drk_last_launch_count() == 0
    torch.cuda.synchronize()
    # W = 0: uniform distribution, logp = -ln V exactly up to rounding
    assert call() == B.DRK_OK
    torch.cuda.synchronize()
    assert torch.allclose(logp, torch.full_like(logp, -math.log(V)), atol=1e-5)
    assert B.drk_last_launch_count() == 2


@pytest.mark.parametrize("T,H,V", [(1, 64, 300), (129, 72, 4099), (300, 512, 257)])
def test_forward_over_usable_rows_at_ragged_sizes(T, H, V):
    case = Hh.build_plain_case(f"fr{T}", T=T, H=H, V=V, dtype=torch.bfloat16, S=3, seed=T + V + 1, mask_frac=0.3)
    dev = run_device(case, make_params(*OPEN, v_chunk=256, forward_rows=1))
    assert dev["status"] == 0
    need = case.loss_mask.numpy().astype(bool)
    got = Hh.f64(dev["logp"])
    if need.any():
        assert np.abs(got[need] - case.logp[need]).max() <= Hh.TOL_LOGP_BF16
    assert (got[~need] == 0).all()
    full = dict(dev)
    full["logp"] = torch.where(torch.from_numpy(need), dev["logp"], torch.from_numpy(case.logp).float())
    full["lse"] = torch.where(torch.from_numpy(need), dev["lse"], torch.from_numpy(case.lse).float())
    del full["entropy"]
    Hh.check_against_oracle(case, full, *OPEN)


def test_forward_rows_with_nothing_usable():
    # every token masked out: no row is evaluated, nothing is retained, gradients are exactly zero
    case = Hh.build_plain_case("fr0", T=200, H=64, V=700, dtype=torch.bfloat16, S=2, seed=77)
    case.loss_mask = torch.zeros_like(case.loss_mask)
    dev = run_device(case, make_params(*OPEN, forward_rows=1))
    assert dev["status"] == 0
    assert (dev["logp"] == 0).all() and (dev["lse"] == 0).all() and (dev["entropy"] == 0).all()
    assert (dev["seg_keep"] == 0).all() and (dev["counters"] == 0).all() and float(dev["loss"]) == 0.0
    assert (dev["dH"] == 0).all() and (dev["dW"] == 0).all()


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_SIMT])
def test_large_logits_stay_finite_and_accurate(engine):
    # logits of magnitude ~100: the running-max subtraction must keep exp() in range on every tile
    case = Hh.build_plain_case("big", T=300, H=512, V=5000, dtype=torch.bfloat16, S=3, seed=91)
    case.hidden = (case.hidden.float() * 8).to(torch.bfloat16)
    case.W = (case.W.float() * 8).to(torch.bfloat16)
    from oracle import drk_oracle as O
    case.s = O.logits(Hh.f64(case.hidden), Hh.f64(case.W))
    assert np.abs(case.s).max() > 80
    case.logp, case.lse = O.token_logprob(case.s, case.ids.numpy())
    case.rollout_logp = torch.from_numpy(case.logp.astype(np.float32))
    dev = run_device(case, make_params(*OPEN, engine=engine, v_chunk=1024))
    assert dev["status"] == 0
    assert torch.isfinite(dev["logp"]).all() and torch.isfinite(dev["dW"]).all() and torch.isfinite(dev["dH"]).all()
    # fp32 accumulation of ~100-sized logits: absolute error scales with the magnitude
    tol = Hh.TOL_LOGP_BF16 * max(1.0, float(np.abs(case.logp).max()) / 10)
    assert np.abs(Hh.f64(dev["logp"]) - case.logp).max() <= tol
    ref = Hh.oracle_eval(case, *OPEN)
    assert Hh.rel_fro(Hh.f64(dev["dH"]), ref["dH"]) <= Hh.TOL_GRAD_FRO
    assert Hh.rel_fro(Hh.f64(dev["dW"]), ref["dW"]) <= Hh.TOL_GRAD_FRO


def test_a_wait_that_runs_out_reports_a_timeout_and_leaves_the_context_usable():
    # a barrier that nothing signals: the bounded wait gives up after its limit, the other waiter of the block
    # leaves on the abort flag long before its own 2 s limit, and the status word says so
    dev = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    waited = torch.zeros(2, dtype=torch.int64, device=dev)
    B.drk_selftest_bounded_wait(50, status, waited)
    torch.cuda.synchronize()
    assert int(status.item()) == B.DRK_STATUS_TIMEOUT
    w = waited.tolist()
    assert 50e6 <= w[0] < 150e6, w            # the limit, not more than a little beyond it
    assert w[1] < 150e6, w                    # the warp did not sit out its own limit
    assert B.drk_selftest_bounded_wait(0, status, waited, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_selftest_bounded_wait(5000, status, waited, check=False) == B.DRK_ERR_INVALID_ARG
    # the context is intact: an ordinary call right after it works
    case = Hh.build_plain_case("after-timeout", T=300, H=64, V=700, dtype=torch.bfloat16, S=2, seed=3)
    logp, lse, st = B.pg_logprob_fwd(case.hidden.to(dev), case.W.to(dev), case.ids.to(dev))
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert float((logp.double().cpu() - torch.from_numpy(case.logp)).abs().max()) <= Hh.TOL_LOGP_BF16


@pytest.mark.parametrize("T,H,V,S", [(200000, 64, 520, 40), (96, 64, 600000, 3)],
                         ids=["many-rows", "wide-vocabulary"])
def test_extreme_aspect_ratios(T, H, V, S):
    # far more row tiles than the benchmark shapes have (index arithmetic past 2^17 rows, hundreds of compaction
    # blocks), and a vocabulary four times the benchmark's with a handful of rows (thousands of vocabulary tiles,
    # dozens of chunks)
    case = Hh.build_plain_case("aspect", T=T, H=H, V=V, dtype=torch.bfloat16, S=S, seed=T % 97, mask_frac=0.25)
    lo, hi = Hh.wide_band(case)
    veto = float(np.float32(1e-4))
    for engine in (B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA):
        dev = run_device(case, make_params(lo, hi, veto, engine=engine, dh_dtype=B.DRK_BF16))
        assert dev["status"] == 0
        Hh.check_against_oracle(case, dev, lo, hi, veto)


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA])
def test_steady_state_calls_encode_no_tensor_maps(engine):
    # tensor maps depend on addresses and geometry only: a second call on the same buffers finds all of them
    d = torch.device("cuda:0")
    case = Hh.build_plain_case("maps", T=300, H=128, V=1500, dtype=torch.bfloat16, S=3, seed=31)
    p = make_params(*OPEN, v_chunk=512, engine=engine)
    bufs = B.PgLossBuffers(case.T, case.H, case.V, case.S, B.DRK_BF16, p, d)
    ins = [t.to(d) for t in (case.hidden, case.W, case.ids, case.rollout_logp, case.loss_mask, case.cu, case.seg_adv)]
    B.pg_loss_fwd_bwd(*ins, p, bufs)
    torch.cuda.synchronize()
    first = (bufs.loss.clone(), bufs.dW.clone(), bufs.dH.clone())
    n = B.drk_tensor_map_encodes()
    assert n > 0
    B.pg_loss_fwd_bwd(*ins, p, bufs)
    torch.cuda.synchronize()
    assert B.drk_tensor_map_encodes() == n
    assert torch.equal(bufs.loss, first[0]) and torch.equal(bufs.dW, first[1]) and torch.equal(bufs.dH, first[2])
    # other buffers of the same sizes (new addresses, or recycled ones whose maps are still valid)
    bufs2 = B.PgLossBuffers(case.T, case.H, case.V, case.S, B.DRK_BF16, p, d)
    B.pg_loss_fwd_bwd(*ins, p, bufs2)
    torch.cuda.synchronize()
    assert torch.equal(bufs2.dW, first[1]) and torch.equal(bufs2.dH, first[2])


def test_a_failing_host_step_enqueues_nothing():
    # every tensor map of the forward and of all chunks of the backward is built before the first enqueue: when
    # the k-th request fails (injected on the host), the call reports DRK_ERR_CUDA and neither the outputs nor
    # the status word nor the stream have been touched, whichever map it was
    d = torch.device("cuda:0")
    case = Hh.build_plain_case("inject", T=300, H=128, V=1500, dtype=torch.bfloat16, S=3, seed=32)
    p = make_params(*OPEN, v_chunk=512)          # three chunks: 2 forward maps + 4 + 3 * 4 + 1 backward maps
    ins = [t.to(d) for t in (case.hidden, case.W, case.ids, case.rollout_logp, case.loss_mask, case.cu, case.seg_adv)]
    code = B.DRK_BF16
    for nth in (1, 2, 3, 7, 12, 19):
        bufs = B.PgLossBuffers(case.T, case.H, case.V, case.S, code, p, d)
        for t in (bufs.logp, bufs.lse, bufs.dH, bufs.dW, bufs.loss):
            t.fill_(float("nan"))
        torch.cuda.synchronize()
        B.drk_selftest_fail_tensor_map(nth)
        rc = B.drk_pg_loss_fwd_bwd(ins[0], ins[1], code, ins[2], ins[3], ins[4], ins[5], ins[6], case.T, case.H, case.V,
                                   case.S, p, bufs.loss, bufs.logp, bufs.lse, bufs.entropy, bufs.seg_w, bufs.seg_keep,
                                   bufs.counters, bufs.dH, bufs.dW, bufs.workspace, bufs.workspace_bytes, bufs.status,
                                   check=False)
        B.drk_selftest_fail_tensor_map(0)
        torch.cuda.synchronize()
        assert rc == B.DRK_ERR_CUDA, nth
        assert B.drk_last_launch_count() == 0
        assert int(bufs.status.item()) == 0
        for t in (bufs.logp, bufs.lse, bufs.dH, bufs.dW, bufs.loss):
            assert torch.isnan(t.float()).all(), nth
    # and the next ordinary call is unaffected
    dev = run_device(case, p)
    assert dev["status"] == 0
    Hh.check_against_oracle(case, dev, *OPEN)
