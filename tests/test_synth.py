"""The seeded input generators: determinism and structural validity."""
import torch

from benchlib import synth


def test_rollout_batch_is_deterministic_and_well_formed():
    a = synth.rollout_batch(4, 8, 3, 16, 64, seed=7)
    b = synth.rollout_batch(4, 8, 3, 16, 64, seed=7)
    assert torch.equal(a.reward, b.reward) and torch.equal(a.resp_len, b.resp_len)
    assert a.reward.shape == (32, 3) and (a.valid == 1).all()
    nz = a.reward[a.reward > 0]
    assert ((a.reward == 0).float().mean() > 0.1) and nz.min() > 0 and nz.max() <= 1.5
    assert (a.prompt_of_rollout[1:] >= a.prompt_of_rollout[:-1]).all()


def test_ragged_batch_has_the_degenerate_groups():
    rb = synth.rollout_batch(8, 8, 4, 16, 64, seed=3, ragged=True, ctx_frac=0.4)
    assert int(rb.valid[:8, 3].sum()) == 1                       # group of one
    assert (rb.reward[8:16] == 1.25).all()                       # all-equal group
    assert (rb.reward[16:24] == 0).all()                         # all-zero group
    assert (rb.reward[rb.valid == 0] == 0).all() and (rb.resp_len[rb.valid == 0] == 0).all()
    v = rb.valid.int()
    assert (v[:, 1:] <= v[:, :-1]).all()                         # termination is final
    frac = rb.ctx_len.sum().item() / (rb.ctx_len.sum().item() + rb.resp_len.sum().item())
    assert 0.35 < frac < 0.45


def test_packing_keeps_whole_segments():
    rb = synth.rollout_batch(4, 8, 3, 16, 128, seed=1, ctx_frac=0.25)
    plans = synth.pack_first_fit(rb, 700)
    total = sum(len(p.segments) for p in plans)
    assert total == int(rb.valid.sum())
    for p in plans:
        assert p.used <= 700
        cu, mask, sr, st = synth.plan_tensors(p, lead_pad=0)
        assert cu[0] == 0 and cu[-1] == p.used and (cu[1:] >= cu[:-1]).all()
        assert int(mask.sum()) == sum(s.resp for s in p.segments)
        assert (mask[p.used:] == 0).all()
    eq = synth.equal_segments_plan(4096, 8, 3)
    assert eq.used == 4096 and len(eq.segments) == 24


def test_dense_operands_and_draws():
    h, W, row_of = synth.dense_operands(64, 32, 100, torch.bfloat16, seed=5)
    h2, W2, _ = synth.dense_operands(64, 32, 100, torch.bfloat16, seed=5)
    assert torch.equal(h, h2) and torch.equal(W, W2) and row_of is None
    assert 0.015 < W.float().std() < 0.025 and 0.9 < h.float().std() < 1.1
    h, W, row_of = synth.dense_operands(64, 32, 100, torch.float32, seed=5, distinct_rows=4)
    assert torch.unique(h, dim=0).shape[0] <= 4 and row_of.shape == (64,)
    cu = torch.tensor([0, 500, 1000], dtype=torch.int32)
    u, noise = synth.token_draws(1000, 3, sigma=0.1, outlier_frac=0.01, outlier_segments=torch.tensor([1]),
                                 cu_seqlens=cu)
    assert (noise[:500].abs() < 1.0).all() and (noise[500:].abs() >= 2.0).sum() >= 3
    assert u.min() >= 0 and u.max() < 1


def test_threshold_between_never_sits_on_a_value():
    import random
    rnd = random.Random(3)
    for n in (2, 3, 5, 6, 16, 19, 28, 33):
        vals = [rnd.random() for _ in range(n)]
        q = synth.threshold_between(vals)
        assert all(abs(q - v) > 0 for v in vals)
        below = sum(v < q for v in vals)
        assert 0 < below < n and abs(below - n / 2) <= max(1.5, 0.2 * n)      # about half on either side
        gaps = sorted(vals)
        lo = max(v for v in vals if v < q)
        hi = min(v for v in vals if v > q)
        assert abs(q - 0.5 * (lo + hi)) < 1e-15                                # midway between its neighbours
    assert synth.threshold_between([]) > 0 and synth.threshold_between([0.25]) == 0.5


def test_nudged_samples_land_inside_the_paper_band_with_margin():
    # the input recipe of the parity tests: a seeded 15 % of the clean samples get a mean log-ratio inside
    # +-6e-4, at least 4e-4 away from the edges ln 0.999 / ln 1.001; samples with outlier tokens are left alone
    import math
    import numpy as np
    from tests import helpers as Hh
    rng = np.random.default_rng(0)
    S, L = 20, 200
    cu = np.arange(0, (S + 1) * L, L)
    T = S * L
    logp = -rng.random(T) * 8
    noise = rng.normal(0, 0.1, T)
    noise[3 * L + 5] = -9.5                    # an outlier token in sample 3
    mask = (rng.random(T) < 0.9).astype(np.uint8)
    rl = (logp + noise).astype(np.float32)
    out = Hh.nudge_into_band(logp, rl, mask, cu, seed=1)
    assert out.dtype == np.float32
    moved = []
    for g in range(S):
        sel = mask[cu[g]:cu[g + 1]].astype(bool)
        before = (logp[cu[g]:cu[g + 1]] - rl[cu[g]:cu[g + 1]].astype(np.float64))[sel].mean()
        after = (logp[cu[g]:cu[g + 1]] - out[cu[g]:cu[g + 1]].astype(np.float64))[sel].mean()
        if abs(before - after) > 1e-9:
            moved.append(g)
            assert abs(after) <= 6e-4 + 1e-6
            assert min(abs(after - math.log(0.999)), abs(after - math.log(1.001))) >= 3.9e-4
            # unmasked tokens are untouched
            assert np.array_equal(out[cu[g]:cu[g + 1]][~sel], rl[cu[g]:cu[g + 1]][~sel])
    assert len(moved) == max(2, round(0.15 * 19)) and 3 not in moved
