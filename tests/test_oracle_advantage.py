"""Pins for the oracle's returns and advantages (Sec. 4.2, Eq. 2, 3, 5)."""
import itertools
import os

import numpy as np
import pytest

from oracle import drk_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_numbers(name):
    vals = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                vals.append(float(line))
    return vals


def test_worked_three_turn_example():
    # Speedups printed for the LayerNorm case (App. E): all turns correct, so
    # Eq. 1 gives R = 1 + speedup, and Eq. 2 with gamma = 1 gives suffix sums.
    sp = _read_numbers("layernorm_case_speedups.txt")
    assert sp == [1.04, 1.21, 1.45]
    R = np.array([[1.0 + min(s, 3.0) for s in sp]])
    G = O.returns(R, np.ones((1, 3), dtype=np.uint8), gamma=1.0)
    assert np.allclose(G[0], [6.70, 4.66, 2.45], atol=1e-12)


def test_gamma_special_cases():
    rng = np.random.default_rng(0)
    R = rng.uniform(0, 4, size=(5, 4))
    valid = np.ones((5, 4), dtype=np.uint8)
    # gamma = 1: plain suffix sums
    G1 = O.returns(R, valid, 1.0)
    assert np.allclose(G1, np.cumsum(R[:, ::-1], axis=1)[:, ::-1], atol=1e-13)
    # gamma = 0: the reward itself (0**0 = 1)
    G0 = O.returns(R, valid, 0.0)
    assert np.array_equal(G0, R)
    # general gamma against Horner's recurrence, an independent evaluation order
    g = 0.7
    Gg = O.returns(R, valid, g)
    ref = np.zeros_like(R)
    acc = np.zeros(5)
    for t in range(3, -1, -1):
        acc = R[:, t] + g * acc
        ref[:, t] = acc
    assert np.allclose(Gg, ref, atol=1e-13)


def test_returns_skip_invalid_turns():
    R = np.array([[1.0, 2.0, 4.0, 8.0]])
    valid = np.array([[1, 0, 1, 0]], dtype=np.uint8)
    G = O.returns(R, valid, 0.5)
    # turn 0 sees turn 2 at distance 2; invalid turns give 0 and contribute nothing
    assert np.allclose(G[0], [1.0 + 0.25 * 4.0, 0.0, 4.0, 0.0])


def test_hand_example_sparse_success():
    # one success among four: TRLOO gives it the full gap, GRPO shrinks it
    G = np.array([[0.0], [0.0], [0.0], [4.0]])
    valid = np.ones((4, 1), dtype=np.uint8)
    prompt = np.zeros(4, dtype=np.int32)
    A, N = O.trloo_advantage(G, valid, prompt)
    assert np.allclose(A[:, 0], [-4 / 3, -4 / 3, -4 / 3, 4.0], atol=1e-15)
    assert (N == 4).all()
    Ag, _ = O.grpo_advantage(G, valid, prompt)
    assert np.allclose(Ag[:, 0], [-1, -1, -1, 3], atol=1e-15)


def _random_case(rng, P, K, Tmax, p_valid=0.8):
    R = P * K
    reward = rng.uniform(0, 4, size=(R, Tmax))
    valid = (rng.uniform(size=(R, Tmax)) < p_valid).astype(np.uint8)
    prompt = np.repeat(np.arange(P, dtype=np.int32), K)
    return reward, valid, prompt


def test_closed_form_and_grpo_ratio():
    rng = np.random.default_rng(1)
    for _ in range(20):
        reward, valid, prompt = _random_case(rng, P=3, K=6, Tmax=3)
        G = O.returns(reward, valid, 1.0)
        A, N = O.trloo_advantage(G, valid, prompt)
        Ag, Ng = O.grpo_advantage(G, valid, prompt)
        assert np.array_equal(N, Ng)
        m = N > 1
        # Eq. 5's equivalent form: A_TRLOO = N/(N-1) (G - mean) = N/(N-1) A_GRPO
        assert np.allclose(A[m], N[m] / (N[m] - 1) * Ag[m], atol=1e-12)
        # groups of one: TRLOO 0 (documented reading), GRPO 0 by definition
        assert (A[N == 1] == 0).all() and (Ag[N == 1] == 0).all()
        assert (A[N == 0] == 0).all()
        # advantages sum to zero inside every (prompt, turn) group
        for p in range(3):
            rows = prompt == p
            for t in range(3):
                sel = rows & (valid[:, t] > 0)
                if sel.sum() > 1:
                    assert abs(A[sel, t].sum()) < 1e-12
                    assert abs(Ag[sel, t].sum()) < 1e-12


def test_brute_force_double_loop():
    rng = np.random.default_rng(2)
    reward, valid, prompt = _random_case(rng, P=4, K=5, Tmax=4, p_valid=0.7)
    G = O.returns(reward, valid, 1.0)
    A, N = O.trloo_advantage(G, valid, prompt)
    R = G.shape[0]
    for i, t in itertools.product(range(R), range(4)):
        if not valid[i, t]:
            assert A[i, t] == 0 and N[i, t] == 0
            continue
        others = [G[j, t] for j in range(R) if j != i and prompt[j] == prompt[i] and valid[j, t]]
        assert N[i, t] == len(others) + 1
        exp = G[i, t] - np.mean(others) if others else 0.0
        assert abs(A[i, t] - exp) < 1e-12


def test_perturbation_leave_one_out():
    # raising G_i by d raises A_i by exactly d and lowers every other A_j by d/(N-1)
    G = np.array([[1.0], [2.5], [0.0], [3.0], [1.5]])
    valid = np.ones((5, 1), dtype=np.uint8)
    prompt = np.zeros(5, dtype=np.int32)
    A0, _ = O.trloo_advantage(G, valid, prompt)
    G2 = G.copy()
    G2[1, 0] += 0.75
    A1, _ = O.trloo_advantage(G2, valid, prompt)
    d = A1 - A0
    assert abs(d[1, 0] - 0.75) < 1e-14
    for j in (0, 2, 3, 4):
        assert abs(d[j, 0] + 0.75 / 4) < 1e-14


def test_degenerate_groups():
    valid = np.ones((4, 1), dtype=np.uint8)
    prompt = np.zeros(4, dtype=np.int32)
    A, _ = O.trloo_advantage(np.full((4, 1), 2.0), valid, prompt)
    assert np.abs(A).max() < 1e-15
    # N = 2: A_1 = G_1 - G_2 = -A_2
    G = np.array([[3.0], [1.0]])
    A, N = O.trloo_advantage(G, np.ones((2, 1), dtype=np.uint8), np.zeros(2, dtype=np.int32))
    assert A[0, 0] == 2.0 and A[1, 0] == -2.0 and (N == 2).all()
    # groups never mix prompts
    G = np.array([[3.0], [1.0], [10.0], [20.0]])
    A, _ = O.trloo_advantage(G, np.ones((4, 1), dtype=np.uint8), np.array([0, 0, 1, 1], dtype=np.int32))
    assert np.allclose(A[:, 0], [2, -2, -10, 10])


def test_self_inclusion_shrinkage_monte_carlo():
    # Eq. 4: on a one-step softmax bandit the GRPO estimator's expectation is
    # (1 - 1/N) times the true gradient, TRLOO's equals it.  Exact expectation
    # by enumeration over all N-tuples of actions (N = 3, 3 actions).
    theta = np.array([0.3, -0.2, 0.5])
    pi = np.exp(theta) / np.exp(theta).sum()
    rew = np.array([1.0, 0.0, 2.5])
    # true gradient of J = sum_a pi_a r_a w.r.t. theta
    grad_true = pi * (rew - (pi * rew).sum())
    N = 3
    valid = np.ones((N, 1), dtype=np.uint8)
    prompt = np.zeros(N, dtype=np.int32)
    e_grpo = np.zeros(3)
    e_loo = np.zeros(3)
    for acts in itertools.product(range(3), repeat=N):
        pr = np.prod([pi[a] for a in acts])
        G = np.array([[rew[a]] for a in acts])
        Ag, _ = O.grpo_advantage(G, valid, prompt)
        Al, _ = O.trloo_advantage(G, valid, prompt)
        for i, a in enumerate(acts):
            score = -pi.copy()
            score[a] += 1.0
            e_grpo += pr * score * Ag[i, 0] / N
            e_loo += pr * score * Al[i, 0] / N
    assert np.allclose(e_loo, grad_true, atol=1e-13)
    assert np.allclose(e_grpo, (1 - 1 / N) * grad_true, atol=1e-13)
