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
