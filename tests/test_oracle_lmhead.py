"""Pins for the oracle's log-softmax over the LM head, MRS, loss and gradients."""
import math

import numpy as np
import torch

from oracle import drk_oracle as O


def _tiny(seed=0, T=12, H=8, V=16):
    rng = np.random.default_rng(seed)
    hidden = rng.normal(size=(T, H))
    W = rng.normal(scale=0.5, size=(V, H))
    ids = rng.integers(0, V, size=T)
    return hidden, W, ids


# ----------------------------------------------------------------- log-softmax

def test_zero_weights_uniform():
    hidden, W, ids = _tiny()
    s = O.logits(hidden, np.zeros_like(W))
    logp, lse = O.token_logprob(s, ids)
    assert np.allclose(lse, math.log(16), atol=1e-15)
    assert np.allclose(logp, -math.log(16), atol=1e-15)


def test_logits_operand_order():
    # s[t,v] = <hidden[t], W[v]>: a transposed operand or a swapped index fails
    hidden = np.array([[1.0, 2.0], [0.0, -1.0], [3.0, 0.5]])
    W = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0], [2.0, -1.0]])
    s = O.logits(hidden, W)
    assert s.shape == (3, 4)
    assert np.array_equal(s, [[1, 2, 3, 0], [0, -1, -1, 1], [3, 0.5, 3.5, 5.5]])


def test_two_class_is_logistic():
    rng = np.random.default_rng(3)
    s = rng.normal(scale=3.0, size=(50, 2))
    ids = rng.integers(0, 2, size=50)
    logp, _ = O.token_logprob(s, ids)
    other = s[np.arange(50), 1 - ids]
    own = s[np.arange(50), ids]
    softplus = np.logaddexp(0.0, other - own)
    assert np.allclose(logp, -softplus, atol=1e-13)


def test_shift_invariance_and_normalisation():
    rng = np.random.default_rng(4)
    s = rng.normal(scale=2.0, size=(9, 33))
    ids = rng.integers(0, 33, size=9)
    logp, lse = O.token_logprob(s, ids)
    logp2, lse2 = O.token_logprob(s + 7.25, ids)
    assert np.allclose(logp, logp2, atol=1e-13)
    assert np.allclose(lse2 - lse, 7.25, atol=1e-13)
    allp = np.exp(s - lse[:, None]).sum(axis=1)
    assert np.allclose(allp, 1.0, atol=1e-13)


def test_large_logits_need_max_subtraction():
    s = np.array([[800.0, 799.0, -800.0], [-800.0, -801.0, -802.0]])
    logp, lse = O.token_logprob(s, np.array([0, 2]))
    assert np.all(np.isfinite(lse))
    assert abs(lse[0] - (800.0 + math.log1p(math.exp(-1.0)))) < 1e-12
    assert abs(logp[1] - (-2.0 - math.log(1 + math.exp(-1) + math.exp(-2)))) < 1e-12


def test_against_float64_library_log_softmax():
    hidden, W, ids = _tiny(5, T=20, H=16, V=40)
    s = O.logits(hidden, W)
    logp, lse = O.token_logprob(s, ids)
    ts = torch.from_numpy(hidden) @ torch.from_numpy(W).T
    ref = torch.log_softmax(ts, dim=1)[torch.arange(20), torch.from_numpy(ids)]
    assert np.allclose(logp, ref.numpy(), atol=1e-13)
    assert np.allclose(lse, torch.logsumexp(ts, dim=1).numpy(), atol=1e-13)


def test_chunked_online_logsumexp_equals_one_shot():
    # the running (max, sum) recurrence used by a chunked evaluation reaches
    # the same value as the one-shot definition, for any chunk size
    rng = np.random.default_rng(6)
    s = rng.normal(scale=4.0, size=(7, 301))
    lse = O.logsumexp_rows(s)
    for chunk in (1, 7, 128, 301):
        m = np.full(7, -np.inf)
        l = np.zeros(7)
        for c0 in range(0, 301, chunk):
            blk = s[:, c0:c0 + chunk]
            m2 = np.maximum(m, blk.max(axis=1))
            l = l * np.exp(m - m2) + np.exp(blk - m2[:, None]).sum(axis=1)
            m = m2
        assert np.allclose(m + np.log(l), lse, atol=1e-12)


# ------------------------------------------------------------------------- MRS

def test_mrs_agreeing_logprobs_weight_one():
    logp = -np.random.default_rng(7).uniform(0.1, 5, size=20)
    cu = np.array([0, 8, 20])
    r = O.mrs(logp, logp.copy(), np.ones(20, dtype=np.uint8), cu)
    assert np.all(r.w == 1.0) and r.keep.all() and not r.vetoed.any()


def test_mrs_constant_offset_closed_form():
    logp = -np.linspace(0.5, 3.0, 30)
    cu = np.array([0, 30])
    mask = np.ones(30, dtype=np.uint8)
    for d, keep in [(0.0, True), (9.9e-4, True), (1.0e-3, False), (-1.0e-3, True),
                    (-1.001e-3, False), (0.5, False)]:
        r = O.mrs(logp, logp - d, mask, cu)          # delta = logp - rollout = d
        assert abs(r.w[0] - math.exp(d)) < 1e-12
        assert bool(r.keep[0]) == keep, d
    # the band is closed: w exactly at a bound is retained
    r = O.mrs(np.array([math.log(1.001)]), np.array([0.0]), np.ones(1, np.uint8), np.array([0, 1]))
    assert r.keep[0]


def test_mrs_token_veto():
    L = 100
    logp = np.full(L, -1.0)
    roll = logp.copy()
    roll[17] = -1.0 + 9.3                # this token's ratio is e^-9.3 < 1e-4
    mask = np.ones(L, dtype=np.uint8)
    cu = np.array([0, L])
    r = O.mrs(logp, roll, mask, cu)
    assert r.vetoed[0] and not r.keep[0]
    # with the band switched off only the veto decides
    r = O.mrs(logp, roll, mask, cu, lo=0.0, hi=math.inf)
    assert r.vetoed[0] and not r.keep[0]
    roll[17] = -1.0 + 9.2                # e^-9.2 > 1e-4: no veto
    r = O.mrs(logp, roll, mask, cu, lo=0.0, hi=math.inf)
    assert not r.vetoed[0] and r.keep[0]
    # veto disabled
    roll[17] = -1.0 + 9.3
    r = O.mrs(logp, roll, mask, cu, lo=0.0, hi=math.inf, veto=0.0)
    assert r.keep[0]


def test_mrs_respects_mask_and_segments():
    logp = np.zeros(10)
    roll = np.zeros(10)
    roll[0:3] = 5.0                       # big mismatch, but masked out
    roll[7] = 20.0                        # lies in segment 1 only
    mask = np.array([0, 0, 0, 1, 1, 1, 1, 1, 1, 1], dtype=np.uint8)
    r = O.mrs(logp, roll, mask, np.array([0, 6, 10]))
    assert r.keep[0] and not r.keep[1]
    assert list(r.n_masked) == [3, 4]
    # a segment with no masked token: w = 1, not retained
    r = O.mrs(logp, roll, np.zeros(10, np.uint8), np.array([0, 10]))
    assert r.w[0] == 1.0 and not r.keep[0]


# ------------------------------------------------------------------------ loss

def test_loss_single_segment_closed_form():
    rng = np.random.default_rng(8)
    logp = -rng.uniform(0.1, 4, size=25)
    mask = (rng.uniform(size=25) < 0.7).astype(np.uint8)
    cu = np.array([0, 25])
    r = O.coeff_and_loss(logp, [True], mask, cu, [1.7])
    assert abs(r.loss - (-1.7 * logp[mask > 0].mean())) < 1e-13
    assert r.kept_tokens == int(mask.sum())


def test_loss_linear_zero_and_norm_modes():
    rng = np.random.default_rng(9)
    logp = -rng.uniform(0.1, 4, size=40)
    mask = np.ones(40, np.uint8)
    cu = np.array([2, 12, 30, 38])          # tokens 0,1 and 38,39 are in no segment
    adv = np.array([0.5, -1.0, 2.0])
    keep = np.array([True, False, True])
    r = O.coeff_and_loss(logp, keep, mask, cu, adv)
    assert r.kept_tokens == 18 and r.masked_tokens == 36
    assert (r.coeff[:2] == 0).all() and (r.coeff[38:] == 0).all() and (r.coeff[12:30] == 0).all()
    r2 = O.coeff_and_loss(logp, keep, mask, cu, 3 * adv)
    assert abs(r2.loss - 3 * r.loss) < 1e-13
    rz = O.coeff_and_loss(logp, [False] * 3, mask, cu, adv)
    assert rz.loss == 0.0 and (rz.coeff == 0).all()
    ra = O.coeff_and_loss(logp, keep, mask, cu, adv, norm=O.NORM_ALL_MASKED_TOKENS)
    assert abs(ra.loss - r.loss * 18 / 36) < 1e-13
    re = O.coeff_and_loss(logp, keep, mask, cu, adv, norm=O.NORM_EXPLICIT, explicit_scale=0.125)
    assert abs(re.loss - r.loss * 18 * 0.125) < 1e-13


# ------------------------------------------------------------------- gradients

def _loss_of(hidden, W, ids, coeff):
    logp, _ = O.token_logprob(O.logits(hidden, W), ids)
    return -float(np.sum(coeff * logp))


def test_gradients_match_finite_differences():
    hidden, W, ids = _tiny(10)
    rng = np.random.default_rng(11)
    coeff = rng.normal(size=12)
    coeff[3] = 0.0
    s = O.logits(hidden, W)
    _, lse = O.token_logprob(s, ids)
    dH, dW = O.gradients(hidden, W, s, lse, ids, coeff)
    eps = 1e-5
    for _ in range(25):
        t, h = rng.integers(0, 12), rng.integers(0, 8)
        hp, hm = hidden.copy(), hidden.copy()
        hp[t, h] += eps
        hm[t, h] -= eps
        fd = (_loss_of(hp, W, ids, coeff) - _loss_of(hm, W, ids, coeff)) / (2 * eps)
        assert abs(fd - dH[t, h]) <= 1e-6 * max(1.0, abs(fd))
        v = rng.integers(0, 16)
        Wp, Wm = W.copy(), W.copy()
        Wp[v, h] += eps
        Wm[v, h] -= eps
        fd = (_loss_of(hidden, Wp, ids, coeff) - _loss_of(hidden, Wm, ids, coeff)) / (2 * eps)
        assert abs(fd - dW[v, h]) <= 1e-6 * max(1.0, abs(fd))
    assert (dH[3] == 0).all()


def test_gradient_invariants_and_zero_weight_closed_form():
    hidden, W, ids = _tiny(12)
    coeff = np.random.default_rng(13).normal(size=12)
    s = O.logits(hidden, W)
    _, lse = O.token_logprob(s, ids)
    dL = O.dlogits(s, lse, ids, coeff)
    # score-function identity: every row of softmax - onehot sums to zero
    assert np.allclose(dL.sum(axis=1), 0, atol=1e-14)
    assert np.all(np.sign(dL[np.arange(12), ids]) == -np.sign(coeff))
    dH, dW = O.gradients(hidden, W, s, lse, ids, coeff)
    assert np.allclose(dW.sum(axis=0), 0, atol=1e-13)
    # W = 0: softmax uniform, dH = 0, dW[v] = sum_t c_t (1/V - [v = ids_t]) hidden[t]
    W0 = np.zeros_like(W)
    s0 = O.logits(hidden, W0)
    _, lse0 = O.token_logprob(s0, ids)
    dH0, dW0 = O.gradients(hidden, W0, s0, lse0, ids, coeff)
    assert np.allclose(dH0, 0, atol=1e-15)
    exp = np.zeros_like(W)
    for t in range(12):
        for v in range(16):
            exp[v] += coeff[t] * (1 / 16 - (1.0 if v == ids[t] else 0.0)) * hidden[t]
    assert np.allclose(dW0, exp, atol=1e-13)


def test_full_path_composition():
    hidden, W, ids = _tiny(14, T=24)
    rng = np.random.default_rng(15)
    s = O.logits(hidden, W)
    logp, _ = O.token_logprob(s, ids)
    roll = logp.copy()
    roll[12:] += 0.3                         # second segment falls outside the band
    mask = np.ones(24, np.uint8)
    cu = np.array([0, 12, 24])
    adv = np.array([1.5, -2.0])
    out = O.pg_loss_fwd_bwd(hidden, W, ids, roll, mask, cu, adv)
    assert list(out["keep"]) == [True, False]
    assert out["kept_tokens"] == 12
    assert abs(out["loss"] - (-1.5 * logp[:12].mean())) < 1e-13
    assert (out["dH"][12:] == 0).all()
    # overriding the decision re-evaluates loss and gradients with it
    out2 = O.pg_loss_fwd_bwd(hidden, W, ids, roll, mask, cu, adv, keep_override=[True, True])
    assert out2["kept_tokens"] == 24 and np.abs(out2["dH"][12:]).max() > 0
    # finite-difference check through the composed path, c_t held constant
    eps = 1e-5
    hp, hm = hidden.copy(), hidden.copy()
    hp[2, 5] += eps
    hm[2, 5] -= eps
    fd = (_loss_of(hp, W, ids, out["coeff"]) - _loss_of(hm, W, ids, out["coeff"])) / (2 * eps)
    assert abs(fd - out["dH"][2, 5]) < 1e-7
