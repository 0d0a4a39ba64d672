"""Device path against the oracle, element by element, on the tiny config and on reduced-T versions of
the 8B-, 14B- and ragged-shaped configs (same H, V, dtype and structure; T spans several row tiles and
ends in a ragged one)."""
import math

import numpy as np
import pytest
import torch

from oracle import drk_oracle as O
from paper_2602_05885_b200 import binding as B
from tests import helpers as Hh
from tests.gpu_utils import make_params, run_device

pytestmark = pytest.mark.gpu

F32 = lambda x: float(np.float32(x))
PAPER = (F32(0.999), F32(1.001), F32(1e-4))


def _case_tiny(seed):
    # 2 prompts x 4 rollouts x 2 turns x 64 response tokens, fp32
    return Hh.build_case(f"tiny{seed}", H=256, V=4096, dtype=torch.float32, P=2, K=4, Tmax=2, len_lo=64, len_hi=64,
                         capacity=1024, seed=seed, sigma=0.05)


CASES = {
    "tiny0": lambda: _case_tiny(0),
    "tiny1": lambda: _case_tiny(1),
    "tiny2": lambda: _case_tiny(2),
    # 8B-shaped: lengths scaled down 8x so that a 700-token micro-batch holds whole segments
    "q8b": lambda: Hh.build_case("q8b", H=4096, V=151936, dtype=torch.bfloat16, P=16, K=8, Tmax=3, len_lo=16,
                                 len_hi=128, capacity=700, seed=1000, sigma=0.05),
    # 14B-shaped: mismatch noise 0.1, 1 % outliers concentrated in 10 % of the segments
    "q14b": lambda: Hh.build_case("q14b", H=5120, V=151936, dtype=torch.bfloat16, P=32, K=8, Tmax=3, len_lo=32,
                                  len_hi=256, capacity=650, seed=2000, sigma=0.1, outlier_frac=0.01),
    # ragged multi-turn: 4 turns, early termination, 40 % unmasked context, padding in front and behind
    "ragged": lambda: Hh.build_case("ragged", H=5120, V=151936, dtype=torch.bfloat16, P=32, K=8, Tmax=4, len_lo=16,
                                    len_hi=96, capacity=600, seed=3000, sigma=0.1, outlier_frac=0.01, ragged=True,
                                    ctx_frac=0.4, lead_pad=5),
    # several waves of work units per SM and several vocabulary chunks
    "medium": lambda: Hh.build_case("medium", H=1024, V=8200, dtype=torch.bfloat16, P=16, K=8, Tmax=3, len_lo=64,
                                    len_hi=512, capacity=5000, seed=4000, sigma=0.05),
}
_cache = {}


def get_case(name):
    if name not in _cache:
        if len(_cache) >= 2:            # the big cases hold GBs of oracle logits
            _cache.pop(next(iter(_cache)))
        _cache[name] = CASES[name]()
    return _cache[name]


@pytest.mark.parametrize("name", ["tiny0", "tiny1", "tiny2"])
def test_tiny_fp32(name):
    case = get_case(name)
    for (lo, hi, veto) in (PAPER, Hh.wide_band(case) + (PAPER[2],), (0.0, math.inf, 0.0)):
        dev = run_device(case, make_params(lo, hi, veto))
        assert dev["status"] == 0
        Hh.check_against_oracle(case, dev, lo, hi, veto, paper_decisive=(lo, hi, veto) == PAPER)


def test_tiny_forward_only_and_determinism():
    case = get_case("tiny0")
    d = torch.device("cuda:0")
    a = B.pg_logprob_fwd(case.hidden.to(d), case.W.to(d), case.ids.to(d))
    b = B.pg_logprob_fwd(case.hidden.to(d), case.W.to(d), case.ids.to(d))
    torch.cuda.synchronize()
    assert np.abs(Hh.f64(a[0]) - case.logp).max() <= Hh.TOL_LOGP_F32
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert int(a[2].item()) == 0


@pytest.mark.parametrize("name", ["medium", "q8b", "q14b", "ragged"])
@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA, B.DRK_ENGINE_SIMT])
def test_bf16_shapes(name, engine):
    if engine == B.DRK_ENGINE_SIMT and name in ("q14b", "ragged"):
        pytest.skip("FFMA cross-check runs on two bf16 shapes only (time)")
    case = get_case(name)
    wide = Hh.wide_band(case)
    for (lo, hi, veto) in (PAPER, wide + (PAPER[2],)):
        dev = run_device(case, make_params(lo, hi, veto, engine=engine, v_chunk=2048 if name == "medium" else 0))
        assert dev["status"] == 0
        # under the paper's constants every case holds clearly retained and clearly rejected samples
        ref = Hh.check_against_oracle(case, dev, lo, hi, veto, paper_decisive=(lo, hi, veto) == PAPER)
        if (lo, hi) == wide:
            assert 0 < ref["kept_segs"] < case.S        # both retained and rejected samples present


def test_bf16_output_dtypes_accumulate_and_norms():
    case = get_case("medium")
    lo, hi = Hh.wide_band(case)
    veto = PAPER[2]
    # bf16 gradients
    dev = run_device(case, make_params(lo, hi, veto, dw_dtype=B.DRK_BF16, dh_dtype=B.DRK_BF16, v_chunk=4096))
    Hh.check_against_oracle(case, dev, lo, hi, veto)
    # dW accumulation on top of existing values, fp32 and bf16
    g = torch.Generator().manual_seed(5)
    init = (torch.randn((case.V, case.H), generator=g) * 1e-4)
    for dt, tdt in ((B.DRK_F32, torch.float32), (B.DRK_BF16, torch.bfloat16)):
        init_t = init.to(tdt)
        dev = run_device(case, make_params(lo, hi, veto, dw_dtype=dt, dw_accumulate=1), dW_init=init_t)
        Hh.check_against_oracle(case, dev, lo, hi, veto, dW_before=Hh.f64(init_t))
    # other normalisations
    dev = run_device(case, make_params(lo, hi, veto, norm=B.DRK_NORM_ALL_MASKED_TOKENS))
    Hh.check_against_oracle(case, dev, lo, hi, veto, norm=1)
    dev = run_device(case, make_params(lo, hi, veto, norm=B.DRK_NORM_EXPLICIT, explicit_scale=F32(1 / 4096)))
    Hh.check_against_oracle(case, dev, lo, hi, veto, norm=2, explicit_scale=F32(1 / 4096))


def test_end_to_end_with_device_advantages():
    # advantages from drk_trloo_advantage feed the device loss; the oracle uses its own
    case = get_case("q8b")
    d = torch.device("cuda:0")
    rb = case.rb
    _, adv, _ = B.trloo_advantage(rb.reward.to(d), rb.valid.to(d), rb.prompt_of_rollout.to(d))
    seg_adv_dev = adv[case.seg_rollout.to(d), case.seg_turn.to(d)].contiguous().cpu()
    lo, hi = Hh.wide_band(case)
    dev = run_device(case, make_params(lo, hi, PAPER[2]), seg_adv=seg_adv_dev)
    Hh.check_against_oracle(case, dev, lo, hi, PAPER[2])


def test_keep_flags_from_the_caller():
    # the caller decides retention (e.g. samples split over micro-batches): seg_keep is an input
    case = get_case("medium")
    g = torch.Generator().manual_seed(3)
    keep_in = (torch.rand(case.S, generator=g) < 0.6).to(torch.uint8)
    dev = run_device(case, make_params(*PAPER, keep_from_caller=1), keep_in=keep_in)
    assert torch.equal(dev["seg_keep"], keep_in)
    ref = Hh.oracle_eval(case, *PAPER, keep_override=keep_in.numpy())
    assert dev["counters"][0] == ref["kept_tokens"] and dev["counters"][2] == ref["kept_segs"] == int(keep_in.sum())
    denom = max(abs(ref["loss"]), 1e-3 * float(np.sum(np.abs(ref["coeff"] * case.logp))))
    assert abs(float(dev["loss"]) - ref["loss"]) / denom <= Hh.TOL_LOSS_REL
    assert Hh.rel_fro(Hh.f64(dev["dH"]), ref["dH"]) <= Hh.TOL_GRAD_FRO
    assert Hh.rel_fro(Hh.f64(dev["dW"]), ref["dW"]) <= Hh.TOL_GRAD_FRO
    # seg_w is still this micro-batch's geometric-mean ratio
    assert np.abs(np.log(Hh.f64(dev["seg_w"])) - ref["mrs"].mean_delta).max() <= Hh.TOL_MRS_MEAN


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA])
def test_forward_over_usable_rows_only(engine):
    # ragged case: 40 % context tokens and padding in front and behind; their rows are not evaluated
    case = get_case("ragged")
    lo, hi = Hh.wide_band(case)
    veto = PAPER[2]
    dev = run_device(case, make_params(lo, hi, veto, engine=engine, forward_rows=1))
    assert dev["status"] == 0
    need = np.zeros(case.T, dtype=bool)
    cu = case.cu.numpy()
    for j in range(case.S):
        need[cu[j]:cu[j + 1]] = True
    need &= case.loss_mask.numpy().astype(bool)
    assert 0 < need.sum() < case.T
    for k, ref in (("logp", case.logp), ("lse", case.lse), ("entropy", O.token_entropy(case.s))):
        got = Hh.f64(dev[k])
        assert np.abs(got[need] - ref[need]).max() <= Hh.TOL_LOGP_BF16, k
        assert (got[~need] == 0).all(), k
    # everything downstream only ever reads the usable rows: same decisions, loss and gradients
    full = dict(dev)
    for k, ref in (("logp", case.logp), ("lse", case.lse)):
        full[k] = torch.where(torch.from_numpy(need), dev[k], torch.from_numpy(ref).float())
    del full["entropy"]
    Hh.check_against_oracle(case, full, lo, hi, veto)


def test_dw_chunk_events_mark_finished_slices():
    # a communication stream may start on a slice of dW as soon as its event has fired
    case = get_case("medium")
    d = torch.device("cuda:0")
    p = make_params(0.0, math.inf, 0.0, v_chunk=2048)
    n_chunks, vc = B.drk_pg_bwd_chunks(case.T, case.H, case.V, B.DRK_BF16, p)
    assert vc == 2048 and n_chunks == math.ceil(case.V / 2048) > 1
    events = [torch.cuda.Event() for _ in range(n_chunks)]
    for e in events:
        e.record()                      # creates the underlying cudaEvent_t
    B.set_dw_chunk_events(p, [e.cuda_event for e in events])
    bufs = B.PgLossBuffers(case.T, case.H, case.V, case.S, B.DRK_BF16, p, d)
    bufs.dW.fill_(float("nan"))
    snap = torch.zeros_like(bufs.dW)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    B.pg_loss_fwd_bwd(case.hidden.to(d), case.W.to(d), case.ids.to(d), case.rollout_logp.to(d), case.loss_mask.to(d),
                      case.cu.to(d), case.seg_adv.to(d), p, bufs)
    with torch.cuda.stream(side):
        for i, e in enumerate(events):
            side.wait_event(e)
            a, b = i * vc, min(case.V, (i + 1) * vc)
            snap[a:b].copy_(bufs.dW[a:b], non_blocking=True)
    torch.cuda.synchronize()
    assert torch.isfinite(snap).all() and torch.equal(snap, bufs.dW)
    ref = Hh.oracle_eval(case, 0.0, math.inf, 0.0)
    assert Hh.rel_fro(Hh.f64(bufs.dW), ref["dW"]) <= Hh.TOL_GRAD_FRO
    # a wrong event count is rejected before anything is enqueued
    B.set_dw_chunk_events(p, [e.cuda_event for e in events[:-1]])
    rc = B.drk_pg_loss_fwd_bwd(case.hidden.to(d), case.W.to(d), B.DRK_BF16, case.ids.to(d), case.rollout_logp.to(d),
                               case.loss_mask.to(d), case.cu.to(d), case.seg_adv.to(d), case.T, case.H, case.V, case.S,
                               p, bufs.loss, bufs.logp, bufs.lse, None, bufs.seg_w, bufs.seg_keep, bufs.counters,
                               bufs.dH, bufs.dW, bufs.workspace, bufs.workspace_bytes, bufs.status, check=False)
    assert rc == B.DRK_ERR_INVALID_ARG


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA])
def test_results_are_reproducible_bit_for_bit(engine):
    # no atomics on the loss path: two calls on the same inputs give identical bits
    case = get_case("medium")
    lo, hi = Hh.wide_band(case)
    p = make_params(lo, hi, PAPER[2], engine=engine, v_chunk=2048, dh_dtype=B.DRK_BF16)
    a = run_device(case, p)
    b = run_device(case, p)
    for k in ("logp", "lse", "entropy", "seg_w", "seg_keep", "loss", "counters", "dH", "dW"):
        assert torch.equal(a[k], b[k]), k
    # which block computes which work unit does not matter either: a fixed assignment gives the same bits
    c = run_device(case, make_params(lo, hi, PAPER[2], engine=engine, v_chunk=2048, dh_dtype=B.DRK_BF16,
                                     schedule=B.DRK_SCHEDULE_STATIC))
    assert c["status"] == 0
    for k in ("logp", "lse", "entropy", "seg_w", "seg_keep", "loss", "counters", "dH", "dW"):
        assert torch.equal(a[k], c[k]), k


def test_caller_retention_combined_with_mrs():
    # PRS-style retention flags from the caller, ANDed with the mismatch rejection decided here
    case = get_case("medium")
    lo, hi = Hh.wide_band(case)
    g = torch.Generator().manual_seed(4)
    retain = (torch.rand(case.S, generator=g) < 0.7).to(torch.uint8)
    dev = run_device(case, make_params(lo, hi, PAPER[2], keep_from_caller=2), keep_in=retain)
    m = Hh.oracle_eval(case, lo, hi, PAPER[2], want_grads=False)["mrs"]
    expect = m.keep & retain.numpy().astype(bool)
    got = dev["seg_keep"].numpy().astype(bool)
    Hh.check_decisions("medium+caller", m, Hh.f64(dev["seg_w"]), got, lo, hi, PAPER[2], Hh.TOL_LOGP_BF16,
                       caller_keep=expect)
    assert not (got & ~retain.numpy().astype(bool)).any()          # never kept against the caller's flag
    assert 0 < got.sum() < m.keep.sum()
    ref = Hh.oracle_eval(case, lo, hi, PAPER[2], keep_override=got)
    assert dev["counters"][0] == ref["kept_tokens"] and dev["counters"][2] == ref["kept_segs"]
    assert Hh.rel_fro(Hh.f64(dev["dH"]), ref["dH"]) <= Hh.TOL_GRAD_FRO
    assert Hh.rel_fro(Hh.f64(dev["dW"]), ref["dW"]) <= Hh.TOL_GRAD_FRO


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_SIMT])
def test_reusing_an_earlier_forward(engine):
    # samples judged on log-probs from a separate forward call: the fused call takes logp and lse as inputs and
    # skips its own forward; everything it returns equals the ordinary call's, bit for bit
    case = get_case("medium")
    lo, hi = Hh.wide_band(case)
    p = make_params(lo, hi, PAPER[2], engine=engine, v_chunk=2048)
    whole = run_device(case, p)
    d = torch.device("cuda:0")
    logp, lse, st = B.pg_logprob_fwd(case.hidden.to(d), case.W.to(d), case.ids.to(d), engine=engine)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.equal(logp.cpu(), whole["logp"])
    again = run_device(case, make_params(lo, hi, PAPER[2], engine=engine, v_chunk=2048, reuse_forward=1),
                       logp_in=logp, lse_in=lse)
    for name in ("logp", "lse", "seg_w", "seg_keep", "counters", "loss", "dH", "dW"):
        assert torch.equal(again[name], whole[name]), name
    assert again["launches"] == whole["launches"] - 2           # no forward kernel, no merge
    Hh.check_against_oracle(case, {k: v for k, v in again.items() if k != "entropy"}, lo, hi, PAPER[2])
    # a restricted forward makes no sense together with no forward
    bad = make_params(lo, hi, PAPER[2], reuse_forward=1, forward_rows=1)
    assert B.drk_pg_workspace_bytes(case.T, case.H, case.V, case.S, B.DRK_BF16, bad, 1) == 0


def test_gradient_accumulation_over_the_micro_batches_of_one_rollout_batch():
    # TRLOO once over the whole rollout batch (on the device), then every packed micro-batch through the fused
    # call with dW accumulating and one explicit normaliser for all of them, as a trainer would do; the
    # accumulated dW must match the sum of the oracle's per-micro-batch gradients, the losses add up likewise
    d = torch.device("cuda:0")
    kw = dict(H=512, V=4200, dtype=torch.bfloat16, P=6, K=4, Tmax=3, len_lo=32, len_hi=200, capacity=900, seed=77,
              sigma=0.05)
    from benchlib import synth
    rb = synth.rollout_batch(kw["P"], kw["K"], kw["Tmax"], kw["len_lo"], kw["len_hi"], kw["seed"])
    n_mb = len(synth.pack_first_fit(rb, kw["capacity"]))
    assert n_mb >= 3
    cases = [Hh.build_case(f"mb{i}", microbatch=i, **kw) for i in range(n_mb)]
    _, adv, _ = B.trloo_advantage(rb.reward.to(d), rb.valid.to(d), rb.prompt_of_rollout.to(d))
    scale = F32(1.0 / sum(int(c.loss_mask.sum()) for c in cases))
    open_band = (0.0, math.inf, 0.0)
    dW_acc = torch.zeros((kw["V"], kw["H"]), dtype=torch.float32)
    dW_ref = np.zeros((kw["V"], kw["H"]))
    loss_dev = loss_ref = 0.0
    for c in cases:
        # every micro-batch uses the same W (the generator draws it from the seed alone)
        assert torch.equal(c.W, cases[0].W)
        seg_adv = torch.empty(c.S, dtype=torch.float32, device=d)
        st = torch.zeros(1, dtype=torch.int32, device=d)
        B.drk_segment_advantages(adv, c.seg_rollout.to(torch.int32).to(d), c.seg_turn.to(torch.int32).to(d),
                                 adv.shape[0], adv.shape[1], c.S, seg_adv, st)
        p = make_params(*open_band, norm=B.DRK_NORM_EXPLICIT, explicit_scale=scale, dw_accumulate=1, v_chunk=2048)
        dev = run_device(c, p, seg_adv=seg_adv.cpu(), dW_init=dW_acc)
        assert dev["status"] == 0 and int(st.item()) == 0
        ref = Hh.check_against_oracle(c, dev, *open_band, norm=2, explicit_scale=scale, seg_adv=seg_adv.cpu(),
                                      dW_before=Hh.f64(dW_acc))
        dW_acc = dev["dW"]
        dW_ref += ref["dW"]
        loss_dev += float(dev["loss"])
        loss_ref += ref["loss"]
    assert Hh.rel_fro(Hh.f64(dW_acc), dW_ref) <= Hh.TOL_GRAD_FRO
    assert abs(loss_dev - loss_ref) <= Hh.TOL_LOSS_REL * max(abs(loss_ref), 1e-3)
