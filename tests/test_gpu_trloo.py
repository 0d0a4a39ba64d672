"""drk_trloo_advantage against the oracle (Sec. 4.2, Eq. 2, 3, 5)."""
import numpy as np
import pytest
import torch

from oracle import drk_oracle as O
from paper_2602_05885_b200 import binding as B
from benchlib import synth
from tests.helpers import TOL_ADV_REL

pytestmark = pytest.mark.gpu


def _run(reward, valid, prompt, gamma, baseline):
    d = torch.device("cuda:0")
    ret, adv, n = B.trloo_advantage(reward.to(d), valid.to(d), prompt.to(d), gamma, baseline)
    torch.cuda.synchronize()
    return ret.cpu().numpy(), adv.cpu().numpy(), n.cpu().numpy()


def _check(reward, valid, prompt, gamma=1.0, baseline=B.DRK_BASELINE_TRLOO):
    g32 = float(np.float32(gamma))
    ret, adv, n = _run(reward, valid, prompt, g32, baseline)
    G = O.returns(reward.numpy(), valid.numpy(), g32)
    fn = O.trloo_advantage if baseline == B.DRK_BASELINE_TRLOO else O.grpo_advantage
    A, N = fn(G, valid.numpy(), prompt.numpy())
    assert np.array_equal(n, N)
    assert np.abs(ret - G).max(initial=0) <= 1e-6 * max(1.0, np.abs(G).max(initial=0))
    # relative to max(1, largest |G| of the group); the group's scale bounds the rounding of adv
    scale = max(1.0, float(np.abs(G).max(initial=0)))
    assert np.abs(adv - A).max(initial=0) <= TOL_ADV_REL * scale
    return ret, adv, n


@pytest.mark.parametrize("cfg", [
    dict(P=2, K=4, Tmax=2, seed=0),          # tiny config
    dict(P=16, K=8, Tmax=3, seed=1000),      # 8B-shaped rollout batch
    dict(P=32, K=8, Tmax=3, seed=2000),      # 14B-shaped rollout batch
    dict(P=16, K=16, Tmax=3, seed=5),        # training group size of the paper
    dict(P=3, K=70, Tmax=5, seed=6),         # groups wider than a warp
])
def test_full_groups(cfg):
    rb = synth.rollout_batch(cfg["P"], cfg["K"], cfg["Tmax"], 8, 16, cfg["seed"])
    _, adv, n = _check(rb.reward, rb.valid, rb.prompt_of_rollout)
    assert (n == cfg["K"]).all()
    # advantages sum to zero inside every (prompt, turn) group
    s = adv.reshape(cfg["P"], cfg["K"], cfg["Tmax"]).sum(axis=1)
    assert np.abs(s).max() < 1e-5


def test_ragged_groups_and_degenerate_cases():
    rb = synth.rollout_batch(32, 8, 4, 8, 16, 3000, ragged=True)
    ret, adv, n = _check(rb.reward, rb.valid, rb.prompt_of_rollout)
    K = 8
    assert n[0, 3] == 1 and adv[0, 3] == 0.0                 # a group of one: zero advantage
    assert (adv[K:2 * K] == 0.0).all()                        # all-equal rewards: exactly zero
    assert (adv[2 * K:3 * K] == 0.0).all()                    # all-zero rewards
    inval = rb.valid.numpy() == 0
    assert (adv[inval] == 0).all() and (ret[inval] == 0).all() and (n[inval] == 0).all()
    assert set(np.unique(n)) >= {0, 1, 2}


@pytest.mark.parametrize("gamma", [0.0, 0.5, 0.9])
def test_discount(gamma):
    rb = synth.rollout_batch(4, 8, 4, 8, 16, 7, ragged=True)
    ret, _, _ = _check(rb.reward, rb.valid, rb.prompt_of_rollout, gamma=gamma)
    if gamma == 0.0:
        assert np.array_equal(ret, rb.reward.numpy())


def test_grpo_baseline_and_ratio():
    rb = synth.rollout_batch(6, 8, 3, 8, 16, 8, ragged=True)
    _, a_g, n = _check(rb.reward, rb.valid, rb.prompt_of_rollout, baseline=B.DRK_BASELINE_GRPO)
    _, a_t, _ = _check(rb.reward, rb.valid, rb.prompt_of_rollout, baseline=B.DRK_BASELINE_TRLOO)
    m = n > 1
    assert np.allclose(a_t[m], a_g[m] * n[m] / (n[m] - 1), atol=2e-6)


def test_irregular_prompt_runs_and_empty():
    # prompt runs of different lengths, ids not consecutive
    prompt = torch.tensor([3, 3, 3, 7, 9, 9, 9, 9, 9, 12, 12], dtype=torch.int32)
    g = torch.Generator().manual_seed(9)
    reward = synth.draw_rewards((11, 3), g)
    valid = (torch.rand((11, 3), generator=g) < 0.8).to(torch.uint8)
    _check(reward * valid, valid, prompt)
    # R = 0 and Tmax = 0 enqueue nothing and succeed
    d = torch.device("cuda:0")
    e = torch.empty(0, device=d)
    assert B.drk_trloo_advantage(e, e, e, 0, 3, 1.0, 0, e, e, e) == B.DRK_OK
    assert B.drk_last_launch_count() == 0


def test_scattered_rollouts_of_a_prompt_are_flagged():
    # groups are runs of equal prompt ids (Sec. 4.2 groups by prompt): when a prompt's rollouts are not
    # contiguous the run-based grouping would split its turn groups, and the status word says so
    d = torch.device("cuda:0")
    g = torch.Generator().manual_seed(10)
    reward = synth.draw_rewards((6, 2), g).to(d)
    valid = torch.ones((6, 2), dtype=torch.uint8, device=d)
    for prompt, want in (([0, 0, 1, 1, 2, 2], 0), ([0, 0, 1, 1, 0, 0], B.DRK_STATUS_BAD_GROUPS),
                         ([5, 4, 4, 4, 4, 4], B.DRK_STATUS_BAD_GROUPS)):
        st = torch.zeros(1, dtype=torch.int32, device=d)
        B.trloo_advantage(reward, valid, torch.tensor(prompt, dtype=torch.int32, device=d), status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == want, prompt
