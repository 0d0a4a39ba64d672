"""Pins for the oracle's reward front-end (Eq. 1, profiling reward and PRS of Sec. 5.2) and its generator."""
import os

import numpy as np

from oracle import drk_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [l.strip() for l in f if l.strip() and not l.startswith("#")]


def test_philox_known_answers():
    for line in _lines("philox4x32_10_kat.txt"):
        w = [int(x, 16) for x in line.split()]
        assert O.philox4x32_10(w[0:4], w[4:6]) == tuple(w[6:10])


def test_eq1_reward_values_and_range():
    # the three turns of the LayerNorm case (App. E): correct kernels, speedups 1.04, 1.21, 1.45
    sp = [float(x) for x in _lines("layernorm_case_speedups.txt")]
    R = O.speedup_reward([1, 1, 1], sp, [1.0, 1.0, 1.0])
    assert np.allclose(R, [2.04, 2.21, 2.45], atol=1e-12)
    # incorrect -> 0; the speedup term is clipped at 3, so R lies in {0} U [1, 4]
    R = O.speedup_reward([0, 1, 1, 1], [5.0, 5.0, 10.0, 1.0], [1.0, 1.0, 1.0, 1000.0])
    assert R[0] == 0.0 and R[1] == 4.0 and R[2] == 4.0 and abs(R[3] - 1.001) < 1e-12
    # T_ref / T_kernel, not the inverse
    assert abs(O.speedup_reward([1], [2.0], [4.0])[0] - 1.5) < 1e-15
    rng = np.random.default_rng(0)
    R = O.speedup_reward(rng.integers(0, 2, 1000), rng.uniform(0.1, 10, 1000), rng.uniform(0.1, 10, 1000))
    assert ((R == 0) | ((R >= 1) & (R <= 4))).all()
    # profiling reward: + PR for correct kernels only, R <= 5
    R = O.speedup_reward([1, 0], [2.0, 2.0], [1.0, 1.0], pr=[0.8615, 0.8615])
    assert abs(R[0] - 3.8615) < 1e-12 and R[1] == 0.0


def test_prs_probability_closed_form_and_paper_cases():
    lazy, fused = [float(x) for x in _lines("profiling_ratio_cases.txt")]
    p = O.prs_keep_prob([lazy, fused, 0.3, 0.35, 0.4, 0.299])
    assert p[0] == 0.0 and p[1] == 1.0 and p[2] == 0.0 and p[5] == 0.0
    assert abs(p[3] - 0.5) < 1e-6 and abs(p[4] - 1.0) < 1e-6
    # whatever the random draw, the two printed cases are decided
    for seed in range(5):
        keep = O.prs_retain([lazy, fused], seed=seed, offset=seed * 7)
        assert list(keep) == [False, True]
    # hard-threshold variant of the ablation: keep iff PR >= tau
    assert list(O.prs_retain([0.29, 0.3, 0.31, 0.9], mode=O.PRS_HARD)) == [False, True, True, True]
    assert O.prs_retain([0.0, 1.0], mode=O.PRS_OFF).all()


def test_prs_retention_rate_matches_probability():
    # in the probabilistic band the retained fraction approaches p (binomial, 4 sigma)
    n = 4000
    for pr, p in ((0.32, 0.2), (0.35, 0.5), (0.38, 0.8)):
        keep = O.prs_retain(np.full(n, pr, dtype=np.float32), seed=123, offset=5)
        assert abs(keep.mean() - p) < 4 * np.sqrt(p * (1 - p) / n) + 1e-3
    # the draw depends on seed, offset and index, and is reproducible
    a = O.prs_retain(np.full(64, 0.35, dtype=np.float32), seed=1, offset=0)
    b = O.prs_retain(np.full(64, 0.35, dtype=np.float32), seed=1, offset=0)
    c = O.prs_retain(np.full(64, 0.35, dtype=np.float32), seed=2, offset=0)
    d = O.prs_retain(np.full(64, 0.35, dtype=np.float32), seed=1, offset=1)
    assert (a == b).all() and (a != c).any() and (a != d).any()
    u = [float(O.prs_uniform(9, 3, i)) for i in range(2000)]
    assert 0.0 <= min(u) and max(u) < 1.0 and abs(np.mean(u) - 0.5) < 0.03
