"""The path with the LM head split by vocabulary rows: every "rank" (run here one after the other on one
GPU, each on its own row block of W) computes its statistics, the blocks are stacked as an all-gather
would, every rank computes loss and gradient parts, and the parts are put together as the all-reduce
would.  The assembled result must match the oracle's plain definitions like the unsplit call does, and
the per-rank statistics must match the oracle's per-range definitions."""
import math

import numpy as np
import pytest
import torch

from oracle import drk_oracle as O
from paper_2602_05885_b200 import binding as B
from tests import helpers as Hh
from tests.gpu_utils import make_params

pytestmark = pytest.mark.gpu

F32 = lambda x: float(np.float32(x))
VETO = F32(1e-4)


def run_sharded(case, cuts, p, dev=torch.device("cuda:0")):
    T, H, S, V = case.T, case.H, case.S, case.V
    code = B.DRK_F32 if case.dtype == torch.float32 else B.DRK_BF16
    hidden, ids = case.hidden.to(dev), case.ids.to(dev)
    rl, mask, cu, adv = case.rollout_logp.to(dev), case.loss_mask.to(dev), case.cu.to(dev), case.seg_adv.to(dev)
    shards = [case.W[a:b].to(dev).contiguous() for a, b in cuts]
    stats, launches = [], 0
    for (a, b), Wk in zip(cuts, shards):
        n = B.drk_pg_workspace_bytes(T, H, b - a, 0, code, p, 0)
        ws = torch.empty(n, dtype=torch.uint8, device=dev)
        st = torch.full((T, 4), float("nan"), device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        B.drk_pg_shard_stats_fwd(hidden, Wk, code, ids, T, H, b - a, a, V, p.engine, st, ws, n, status)
        launches += B.drk_last_launch_count()
        assert int(status.item()) == 0
        stats.append(st)
    stats_all = torch.stack(stats).contiguous()
    outs = []
    for (a, b), Wk in zip(cuts, shards):
        bufs = B.PgLossBuffers(T, H, b - a, S, code, p, dev)
        bufs.dH.fill_(float("nan"))
        bufs.dW.fill_(float("nan"))
        B.drk_pg_shard_loss_bwd(hidden, Wk, code, ids, stats_all, len(cuts), rl, mask, cu, adv, T, H, b - a, a, V, S,
                                p, bufs.loss, bufs.logp, bufs.lse, bufs.entropy, bufs.seg_w, bufs.seg_keep,
                                bufs.counters, bufs.dH, bufs.dW, bufs.workspace, bufs.workspace_bytes, bufs.status)
        launches += B.drk_last_launch_count()
        torch.cuda.synchronize()
        assert int(bufs.status.item()) == 0
        outs.append(bufs)
    first = outs[0]
    # the forward-only recombination gives the same log-probs, lse and entropy as the loss call
    lp, z, ent = (torch.full((T,), float("nan"), device=dev) for _ in range(3))
    st_word = torch.zeros(1, dtype=torch.int32, device=dev)
    B.drk_pg_shard_merge(stats_all, len(cuts), ids, T, V, lp, z, ent, st_word)
    torch.cuda.synchronize()
    assert int(st_word.item()) == 0
    assert torch.equal(lp, first.logp) and torch.equal(z, first.lse) and torch.equal(ent, first.entropy)
    for o in outs[1:]:        # what is not a gradient is identical on every rank, bit for bit
        for name in ("loss", "logp", "lse", "entropy", "seg_w", "seg_keep", "counters"):
            assert torch.equal(getattr(o, name), getattr(first, name)), name
    dev_out = dict(logp=first.logp.cpu(), lse=first.lse.cpu(), entropy=first.entropy.cpu(), seg_w=first.seg_w.cpu(),
                   seg_keep=first.seg_keep.cpu(), loss=first.loss.cpu(), counters=first.counters.cpu(),
                   dH=sum(o.dH.float() for o in outs).cpu(), dW=torch.cat([o.dW.float() for o in outs]).cpu(),
                   launches=launches)
    return dev_out, stats_all.cpu()


def check_stats(case, cuts, stats_all):
    tol = Hh.TOL_LOGP_F32 if case.dtype == torch.float32 else Hh.TOL_LOGP_BF16
    for k, (a, b) in enumerate(cuts):
        ref = O.shard_stats(case.s, case.ids.numpy(), a, b)
        got = Hh.f64(stats_all[k])
        # compare what does not depend on the reference point: max, log-sum-exp, mean logit under the range's softmax
        assert np.abs(got[:, 0] - ref[:, 0]).max() <= tol
        assert np.abs((got[:, 0] + np.log(got[:, 1])) - (ref[:, 0] + np.log(ref[:, 1]))).max() <= tol
        assert np.abs(got[:, 2] / got[:, 1] - ref[:, 2] / ref[:, 1]).max() <= tol
        assert np.abs(got[:, 3] - ref[:, 3]).max() <= tol
        owns = (case.ids.numpy() >= a) & (case.ids.numpy() < b)
        assert (got[~owns, 3] == 0).all()


CASES = {
    "tiny": lambda: Hh.build_case("tiny0", H=256, V=4096, dtype=torch.float32, P=2, K=4, Tmax=2, len_lo=64, len_hi=64,
                                  capacity=1024, seed=0, sigma=0.05),
    "medium": lambda: Hh.build_case("medium", H=1024, V=8200, dtype=torch.bfloat16, P=16, K=8, Tmax=3, len_lo=64,
                                    len_hi=512, capacity=5000, seed=4000, sigma=0.05),
    "q8b": lambda: Hh.build_case("q8b", H=4096, V=151936, dtype=torch.bfloat16, P=16, K=8, Tmax=3, len_lo=16,
                                 len_hi=128, capacity=700, seed=1000, sigma=0.05),
}
_cache = {}


def get_case(name):
    if name not in _cache:
        _cache.clear()
        _cache[name] = CASES[name]()
    return _cache[name]


@pytest.mark.parametrize("cuts", [((0, 4096),), ((0, 1000), (1000, 1001), (1001, 4096))])
def test_tiny_fp32_in_ranges(cuts):
    case = get_case("tiny")
    lo, hi = Hh.wide_band(case)
    dev, stats_all = run_sharded(case, cuts, make_params(lo, hi, VETO))
    check_stats(case, cuts, stats_all)
    Hh.check_against_oracle(case, dev, lo, hi, VETO)


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA, B.DRK_ENGINE_SIMT])
@pytest.mark.parametrize("cuts", [((0, 4096), (4096, 8200)), ((0, 3000), (3000, 3001), (3001, 8199), (8199, 8200))])
def test_bf16_in_ranges(engine, cuts):
    case = get_case("medium")
    lo, hi = Hh.wide_band(case)
    for dh in (B.DRK_F32, B.DRK_BF16):
        dev, stats_all = run_sharded(case, cuts, make_params(lo, hi, VETO, engine=engine, v_chunk=2048, dh_dtype=dh))
        check_stats(case, cuts, stats_all)
        ref = Hh.check_against_oracle(case, dev, lo, hi, VETO)
        assert 0 < ref["kept_segs"] < case.S


def test_full_vocabulary_in_two_and_eight_ranges():
    from paper_2602_05885_b200 import dp
    case = get_case("q8b")
    lo, hi = Hh.wide_band(case)
    for world in (2, 8):
        cuts = tuple(dp.vocab_shards(case.V, world))
        assert cuts[0][0] == 0 and cuts[-1][1] == case.V and all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
        dev, stats_all = run_sharded(case, cuts, make_params(lo, hi, VETO))
        check_stats(case, cuts, stats_all)
        Hh.check_against_oracle(case, dev, lo, hi, VETO)


def test_one_range_equals_the_unsplit_call():
    from tests.gpu_utils import run_device
    case = get_case("medium")
    lo, hi = Hh.wide_band(case)
    p = make_params(lo, hi, VETO, v_chunk=2048)
    dev, _ = run_sharded(case, ((0, case.V),), p)
    whole = run_device(case, p)
    for name in ("logp", "lse", "entropy", "seg_keep", "counters", "loss", "dH", "dW"):
        assert torch.equal(dev[name], whole[name]), name


def test_ids_outside_the_vocabulary_and_bad_ranges():
    dev = torch.device("cuda:0")
    case = get_case("medium")
    T, H, V, S = case.T, case.H, case.V, case.S
    p = make_params(0.0, math.inf, 0.0, v_chunk=2048)
    ids = case.ids.clone()
    ids[5] = V            # not a token of the vocabulary
    ids[9] = -3
    a, b = 4096, V
    Wk = case.W[a:b].to(dev).contiguous()
    n = B.drk_pg_workspace_bytes(T, H, b - a, 0, B.DRK_BF16, p, 0)
    ws = torch.empty(n, dtype=torch.uint8, device=dev)
    st = torch.empty((T, 4), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    hidden = case.hidden.to(dev)
    B.drk_pg_shard_stats_fwd(hidden, Wk, B.DRK_BF16, ids.to(dev), T, H, b - a, a, V, p.engine, st, ws, n, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0                      # a token of another range is not an error here
    assert float(st[5, 3]) == 0.0 and float(st[9, 3]) == 0.0
    bufs = B.PgLossBuffers(T, H, b - a, S, B.DRK_BF16, p, dev)
    stats_all = st.unsqueeze(0).contiguous()
    B.drk_pg_shard_loss_bwd(hidden, Wk, B.DRK_BF16, ids.to(dev), stats_all, 1, case.rollout_logp.to(dev),
                            case.loss_mask.to(dev), case.cu.to(dev), case.seg_adv.to(dev), T, H, b - a, a, V, S, p,
                            bufs.loss, bufs.logp, bufs.lse, bufs.entropy, bufs.seg_w, bufs.seg_keep, bufs.counters,
                            bufs.dH, bufs.dW, bufs.workspace, bufs.workspace_bytes, bufs.status)
    torch.cuda.synchronize()
    assert int(bufs.status.item()) & B.DRK_STATUS_BAD_ID
    # host-detected: a range that leaves the vocabulary, no ranges, a restricted forward
    args = lambda vb, vt, ns, pp: (hidden, Wk, B.DRK_BF16, ids.to(dev), stats_all, ns, case.rollout_logp.to(dev),
                                   case.loss_mask.to(dev), case.cu.to(dev), case.seg_adv.to(dev), T, H, b - a, vb, vt,
                                   S, pp, bufs.loss, bufs.logp, bufs.lse, bufs.entropy, bufs.seg_w, bufs.seg_keep,
                                   bufs.counters, bufs.dH, bufs.dW, bufs.workspace, bufs.workspace_bytes, bufs.status)
    assert B.drk_pg_shard_loss_bwd(*args(a + 1, V, 1, p), check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_pg_shard_loss_bwd(*args(a, V, 0, p), check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_pg_shard_loss_bwd(*args(-1, V, 1, p), check=False) == B.DRK_ERR_INVALID_ARG
    p2 = make_params(0.0, math.inf, 0.0, v_chunk=2048, forward_rows=1)
    assert B.drk_pg_shard_loss_bwd(*args(a, V, 1, p2), check=False) == B.DRK_ERR_UNSUPPORTED
    assert B.drk_pg_shard_stats_fwd(hidden, Wk, B.DRK_BF16, ids.to(dev), T, H, b - a, a + 1, V, p.engine, st, ws, n,
                                    status, check=False) == B.DRK_ERR_INVALID_ARG


def test_segment_advantages_gather():
    dev = torch.device("cuda:0")
    case = get_case("medium")
    rb = case.rb
    _, A, _ = Hh.oracle_advantages(rb)
    _, adv, _ = B.trloo_advantage(rb.reward.to(dev), rb.valid.to(dev), rb.prompt_of_rollout.to(dev))
    R, Tmax = adv.shape
    sr, stn = case.seg_rollout.to(torch.int32).to(dev), case.seg_turn.to(torch.int32).to(dev)
    out = torch.full((case.S,), float("nan"), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.drk_segment_advantages(adv, sr, stn, R, Tmax, case.S, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out, adv[sr.long(), stn.long()])                  # index work: bit-exact
    ref = O.segment_advantages(A, case.seg_rollout.numpy(), case.seg_turn.numpy())
    scale = max(1.0, float(np.abs(O.returns(rb.reward.numpy(), rb.valid.numpy(), 1.0)).max()))
    assert np.abs(Hh.f64(out) - ref).max() <= Hh.TOL_ADV_REL * scale
    # indices outside the table: zero advantage and a status bit, nothing read out of bounds
    sr[0] = R
    stn[1] = -1
    B.drk_segment_advantages(adv, sr, stn, R, Tmax, case.S, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.DRK_STATUS_BAD_SEGMENTS and float(out[0]) == 0.0 and float(out[1]) == 0.0
    assert B.drk_segment_advantages(adv, sr, stn, R, Tmax, 0, out, status) == B.DRK_OK


def test_partial_sums_of_dh_are_exchanged_in_fp32():
    # eight ranges of the vocabulary: each range's dH is a partial sum.  Summed in fp32 and rounded once at the end
    # the result is closer to the oracle than the sum of parts that were each rounded to bf16 first, which is
    # why the multi-rank helper refuses 16-bit parts
    from paper_2602_05885_b200 import dp
    case = get_case("medium")
    lo, hi = Hh.wide_band(case)
    cuts = tuple(dp.vocab_shards(case.V, 8, align=128))
    errs = {}
    for name, dh in (("fp32 parts", B.DRK_F32), ("bf16 parts", B.DRK_BF16)):
        dev, _ = run_sharded(case, cuts, make_params(lo, hi, VETO, v_chunk=2048, dh_dtype=dh))
        ref = Hh.check_against_oracle(case, dev, lo, hi, VETO)
        errs[name] = Hh.rel_fro(Hh.f64(dev["dH"]), ref["dH"])
    # (what remains with fp32 parts is the bf16 rounding of the dLogits tiles themselves, about 2e-3)
    assert errs["fp32 parts"] < errs["bf16 parts"] <= Hh.TOL_GRAD_FRO
    Hh.report(f"dH over 8 vocabulary ranges, rel. Frobenius error: {errs}")
