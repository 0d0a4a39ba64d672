"""More pins for the oracle, independent of its own formulas:

  * the analytic gradients against reverse-mode differentiation by a float64 library of the surrogate
    -sum_t c_t log softmax(h W^T)[t, ids_t] written directly (App. A's estimator is its gradient);
  * randomised properties of Eq. 2 / 3 / 5 and of the rejection rule of Sec. 5.1 over arbitrary group
    structures, validity patterns and segmentations (hypothesis).
"""
import math

import numpy as np
import torch
from hypothesis import given, settings, strategies as st

from oracle import drk_oracle as O


def test_gradients_against_library_autodiff():
    rng = np.random.default_rng(11)
    T, H, V = 13, 7, 29
    hidden = rng.normal(size=(T, H))
    W = rng.normal(size=(V, H)) * 0.5
    ids = rng.integers(0, V, size=T)
    coeff = rng.normal(size=T)
    coeff[[1, 6]] = 0.0
    h = torch.tensor(hidden, dtype=torch.float64, requires_grad=True)
    w = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    logp = torch.log_softmax(h @ w.T, dim=1)[torch.arange(T), torch.from_numpy(ids)]
    loss = -(torch.tensor(coeff) * logp).sum()
    loss.backward()
    s = O.logits(hidden, W)
    lp, lse = O.token_logprob(s, ids)
    dH, dW = O.gradients(hidden, W, s, lse, ids, coeff)
    # the oracle's dL is d(loss)/d(logits) for loss = -sum c logp: sign and one-hot term included
    assert np.abs(dH - h.grad.numpy()).max() < 1e-12
    assert np.abs(dW - w.grad.numpy()).max() < 1e-12
    assert abs(float(loss.detach()) + float(np.sum(coeff * lp))) < 1e-12
    assert (dH[[1, 6]] == 0).all()


@st.composite
def rollout_tables(draw):
    P = draw(st.integers(1, 4))
    sizes = [draw(st.integers(1, 6)) for _ in range(P)]
    Tmax = draw(st.integers(1, 4))
    R = sum(sizes)
    prompt = np.repeat(np.arange(P), sizes)
    reward = np.array(draw(st.lists(st.floats(0, 5, allow_nan=False, width=32), min_size=R * Tmax, max_size=R * Tmax)),
                      dtype=np.float64).reshape(R, Tmax)
    valid = np.array(draw(st.lists(st.booleans(), min_size=R * Tmax, max_size=R * Tmax))).reshape(R, Tmax)
    gamma = draw(st.sampled_from([0.0, 0.5, 1.0]))
    return reward, valid, prompt, gamma


@settings(max_examples=60, deadline=None)
@given(rollout_tables())
def test_advantage_properties_on_arbitrary_tables(tab):
    reward, valid, prompt, gamma = tab
    G = O.returns(reward, valid, gamma)
    A, N = O.trloo_advantage(G, valid, prompt)
    Ag, Ng = O.grpo_advantage(G, valid, prompt)
    assert np.array_equal(N, Ng)
    assert (G[~valid] == 0).all() and (A[~valid] == 0).all() and (N[~valid] == 0).all()
    # Eq. 2 as a recurrence over the valid turns of a rollout
    R, Tmax = reward.shape
    for i in range(R):
        nxt = 0.0
        dist = 0
        for t in range(Tmax - 1, -1, -1):
            dist += 1
            if valid[i, t]:
                nxt = reward[i, t] + (gamma ** dist if nxt != 0.0 else 0.0) * nxt
                assert abs(G[i, t] - nxt) < 1e-9
                dist = 0
    for t, g in O.turn_groups(valid, prompt):
        n = len(g)
        assert (N[g, t] == n).all()
        assert abs(Ag[g, t].sum()) < 1e-9                             # Eq. 3 is mean-centred
        if n > 1:
            assert abs(A[g, t].sum()) < 1e-9
            assert np.allclose(A[g, t], n / (n - 1) * Ag[g, t], atol=1e-9)      # Eq. 5's closed form
        else:
            assert A[g[0], t] == 0.0


@st.composite
def segmented_logprobs(draw):
    S = draw(st.integers(1, 5))
    lens = [draw(st.integers(0, 9)) for _ in range(S)]
    lead = draw(st.integers(0, 3))
    T = lead + sum(lens) + draw(st.integers(0, 3))
    cu = np.concatenate([[lead], lead + np.cumsum(lens)]).astype(np.int64)
    delta = np.array(draw(st.lists(st.floats(-12, 3, allow_nan=False), min_size=T, max_size=T)))
    mask = np.array(draw(st.lists(st.booleans(), min_size=T, max_size=T)), dtype=np.uint8)
    return cu, delta, mask


@settings(max_examples=80, deadline=None)
@given(segmented_logprobs(), st.sampled_from([(0.999, 1.001, 1e-4), (0.5, 2.0, 1e-4), (0.0, math.inf, 0.0), (0.9, 1.1, 0.0)]))
def test_rejection_rule_on_arbitrary_segmentations(data, consts):
    cu, delta, mask = data
    lo, hi, veto = consts
    T = delta.shape[0]
    rng = np.random.default_rng(T)
    rollout = rng.normal(size=T)
    m = O.mrs(rollout + delta, rollout, mask, cu, lo, hi, veto)
    for g in range(len(cu) - 1):
        d = [delta[t] for t in range(cu[g], cu[g + 1]) if mask[t]]
        if not d:
            assert not m.keep[g] and m.w[g] == 1.0
            continue
        gm = math.exp(sum(d) / len(d))                                 # geometric mean of the token ratios
        assert abs(m.w[g] - gm) <= 1e-9 * max(1.0, gm)
        veto_fires = veto > 0 and min(d) < math.log(veto)
        assert bool(m.vetoed[g]) == veto_fires
        mean = sum(d) / len(d)
        in_band = (lo <= 0 or mean >= math.log(lo) - 1e-12) and (math.isinf(hi) or mean <= math.log(hi) + 1e-12)
        near = any(abs(mean - math.log(x)) < 1e-9 for x in (lo, hi) if 0 < x < math.inf)
        if not near:
            assert bool(m.keep[g]) == (in_band and not veto_fires)
