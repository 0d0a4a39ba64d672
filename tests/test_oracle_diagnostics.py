"""Pins for the oracle's diagnostics: token entropy, perplexities, log-ratio statistics, gradient norms."""
import math

import numpy as np
import torch

from oracle import drk_oracle as O


def test_entropy_closed_forms():
    # uniform distribution: ln V
    s = np.full((3, 50), 1.7)
    assert np.allclose(O.token_entropy(s), math.log(50), atol=1e-13)
    # two classes: -p ln p - q ln q with p = sigmoid(a - b)
    rng = np.random.default_rng(0)
    s = rng.normal(scale=2.0, size=(20, 2))
    p = 1.0 / (1.0 + np.exp(-(s[:, 0] - s[:, 1])))
    ref = -(p * np.log(p) + (1 - p) * np.log(1 - p))
    assert np.allclose(O.token_entropy(s), ref, atol=1e-12)
    # a one-hot distribution (huge gap) has entropy ~ 0; shifts do not matter
    s = np.array([[100.0, 0.0, 0.0], [3.0, 2.0, 1.0]])
    h = O.token_entropy(s)
    assert h[0] < 1e-40 + 1e-12 and np.allclose(O.token_entropy(s + 11.0), h, atol=1e-12)


def test_entropy_against_float64_library():
    rng = np.random.default_rng(1)
    s = rng.normal(scale=1.5, size=(13, 97))
    ref = torch.distributions.Categorical(logits=torch.from_numpy(s)).entropy().numpy()
    assert np.allclose(O.token_entropy(s), ref, atol=1e-12)


def test_diagnostics_closed_forms():
    T = 20
    logp = np.full(T, -2.0)
    rl = np.full(T, -2.5)
    rl[7] = -6.0                                  # |ratio| outlier inside the selection
    rl[0] = 50.0                                  # outside every segment: ignored
    mask = np.ones(T, np.uint8)
    mask[5] = 0
    rl[5] = -40.0                                 # masked out: ignored
    cu = np.array([2, 10, 18])
    ent = np.linspace(1.0, 2.9, T)
    d = O.diagnostics(logp, rl, ent, mask, cu, dH=np.array([[3.0, 4.0]]), dW=np.full((2, 2), 2.0))
    sel = [t for t in range(2, 18) if t != 5]
    assert d["n_tokens"] == len(sel) == 15
    assert abs(d["ppl_train"] - math.exp(2.0)) < 1e-12
    assert abs(d["ppl_rollout"] - math.exp(-np.mean(rl[sel]))) < 1e-12
    assert abs(d["mean_log_ratio"] - np.mean(logp[sel] - rl[sel])) < 1e-13
    assert abs(d["max_abs_log_ratio"] - 4.0) < 1e-13
    assert abs(d["mean_entropy"] - np.mean(ent[sel])) < 1e-13
    assert d["grad_norm_dH"] == 5.0 and d["grad_norm_dW"] == 4.0
    e = O.diagnostics(logp, rl, ent, np.zeros(T, np.uint8), cu)
    assert e["n_tokens"] == 0 and e["ppl_train"] == 1.0 and e["max_abs_log_ratio"] == 0.0
