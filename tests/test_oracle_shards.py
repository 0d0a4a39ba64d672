"""Pins for the oracle's vocabulary-range functions and the segment gather: recombining ranges must
reproduce the one-shot definitions (already pinned elsewhere) exactly, for any partition; closed forms
for constant logits; a hand-computed two-column case."""
import math

import numpy as np
import pytest

from oracle import drk_oracle as O


def _random_problem(seed, T=9, H=6, V=23):
    rng = np.random.default_rng(seed)
    hidden = rng.normal(size=(T, H))
    W = rng.normal(size=(V, H))
    ids = rng.integers(0, V, size=T)
    coeff = rng.normal(size=T)
    coeff[2] = 0.0
    return hidden, W, ids, coeff


@pytest.mark.parametrize("cuts", [(0, 23), (0, 1, 23), (0, 7, 8, 20, 23), tuple(range(24))])
def test_ranges_recombine_to_the_one_shot_definitions(cuts):
    hidden, W, ids, coeff = _random_problem(len(cuts))
    s = O.logits(hidden, W)
    logp, lse = O.token_logprob(s, ids)
    stats = [O.shard_stats(s, ids, a, b) for a, b in zip(cuts[:-1], cuts[1:])]
    lp, z, ent = O.merge_shard_stats(np.stack(stats))
    assert np.abs(lp - logp).max() < 1e-12 and np.abs(z - lse).max() < 1e-12
    assert np.abs(ent - O.token_entropy(s)).max() < 1e-12
    # the target logit is reported by exactly the range that owns the token
    owners = sum((st[:, 3] != 0).astype(int) for st in stats)
    assert (owners <= 1).all()
    dH, dW = O.gradients(hidden, W, s, lse, ids, coeff)
    parts = [O.shard_gradients(hidden, W, s, lse, ids, coeff, a, b) for a, b in zip(cuts[:-1], cuts[1:])]
    assert np.abs(sum(p[0] for p in parts) - dH).max() < 1e-12
    assert np.abs(np.concatenate([p[1] for p in parts]) - dW).max() < 1e-12
    assert (sum(p[0] for p in parts)[2] == 0).all()          # zero coefficient, zero row


def test_constant_logits_closed_form():
    # W = 0: every logit is 0, so a range of width n has m = 0, l = n, r = 0, g = 0
    hidden = np.ones((3, 4))
    W = np.zeros((10, 4))
    s = O.logits(hidden, W)
    st = O.shard_stats(s, [0, 5, 9], 2, 9)
    assert np.array_equal(st, np.array([[0, 7, 0, 0]] * 3, dtype=float))
    lp, z, ent = O.merge_shard_stats(np.stack([O.shard_stats(s, [0, 5, 9], 0, 2), st, O.shard_stats(s, [0, 5, 9], 9, 10)]))
    assert np.allclose(z, math.log(10)) and np.allclose(lp, -math.log(10)) and np.allclose(ent, math.log(10))


def test_two_columns_by_hand():
    # logits (0, ln 3): probabilities 1/4 and 3/4
    s = np.array([[0.0, math.log(3.0)]])
    a = O.shard_stats(s, [1], 0, 1)
    b = O.shard_stats(s, [1], 1, 2)
    assert np.allclose(a, [[0, 1, 0, 0]]) and np.allclose(b, [[math.log(3), 1, math.log(3), math.log(3)]])
    lp, z, ent = O.merge_shard_stats(np.stack([a, b]))
    assert np.allclose(z, math.log(4)) and np.allclose(lp, math.log(0.75))
    assert np.allclose(ent, -(0.25 * math.log(0.25) + 0.75 * math.log(0.75)))


def test_shifted_maxima_do_not_overflow():
    s = np.array([[800.0, -800.0, 799.0]])
    lp, z, _ = O.merge_shard_stats(np.stack([O.shard_stats(s, [2], 0, 1), O.shard_stats(s, [2], 1, 3)]))
    assert np.isfinite(z).all() and np.allclose(z, 800 + math.log1p(math.exp(-1.0)))
    assert np.allclose(lp, 799 - z)


def test_segment_advantages_by_hand():
    A = np.array([[1.0, 2.0, 3.0], [4.0, 5.0, 6.0]])
    out = O.segment_advantages(A, [1, 0, 1, 0], [2, 0, 0, 1])
    assert np.array_equal(out, [6.0, 1.0, 4.0, 2.0])
    assert O.segment_advantages(A, [], []).shape == (0,)
