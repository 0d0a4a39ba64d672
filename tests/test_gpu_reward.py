"""drk_reward against the oracle: Eq. 1, profiling reward, PRS (soft with Philox draws, hard, off)."""
import numpy as np
import pytest
import torch

from oracle import drk_oracle as O
from paper_2602_05885_b200 import binding as B

pytestmark = pytest.mark.gpu


def _inputs(n, seed):
    g = torch.Generator().manual_seed(seed)
    correct = (torch.rand(n, generator=g) < 0.7).to(torch.uint8)
    t_ref = torch.rand(n, generator=g) * 4 + 0.05
    t_kernel = torch.rand(n, generator=g) * 2 + 0.05
    # profiling ratios spread over [0,1] with many inside the probabilistic band [0.3, 0.4)
    pr = torch.where(torch.rand(n, generator=g) < 0.5, 0.3 + 0.1 * torch.rand(n, generator=g), torch.rand(n, generator=g))
    return correct, t_ref.float(), t_kernel.float(), pr.float()


@pytest.mark.parametrize("n", [1, 257, 768, 5000])
@pytest.mark.parametrize("mode", [B.DRK_PRS_OFF, B.DRK_PRS_SOFT, B.DRK_PRS_HARD])
def test_reward_and_retention(n, mode):
    d = torch.device("cuda:0")
    correct, t_ref, t_kernel, pr = _inputs(n, n + mode)
    p = B.drk_reward_params_default()
    assert p.speedup_clip == 3.0 and abs(p.prs_tau - 0.3) < 1e-7 and abs(p.prs_s - 0.1) < 1e-7
    p.use_pr = 1 if mode != B.DRK_PRS_OFF else 0
    p.prs_mode = mode
    p.seed = 0x123456789ABCDEF
    p.offset = (1 << 33) + 17
    reward = torch.empty(n, device=d)
    retain = torch.full((n,), 7, dtype=torch.uint8, device=d)
    B.drk_reward(correct.to(d), t_ref.to(d), t_kernel.to(d), pr.to(d), n, p, reward, retain)
    assert B.drk_last_launch_count() == 1
    torch.cuda.synchronize()
    R = O.speedup_reward(correct.numpy(), t_ref.numpy(), t_kernel.numpy(), pr.numpy() if p.use_pr else None, 3.0)
    assert np.abs(reward.cpu().numpy() - R).max() <= 1e-6 * 5
    keep = O.prs_retain(pr.numpy(), float(p.prs_tau), float(p.prs_s), mode, p.seed, p.offset)
    assert np.array_equal(retain.cpu().numpy().astype(bool), keep)      # bit-exact decisions
    if mode == B.DRK_PRS_SOFT and n >= 768:
        assert 0 < keep.sum() < n


def test_reward_argument_checks():
    d = torch.device("cuda:0")
    z = torch.zeros(8, device=d)
    zb = torch.zeros(8, dtype=torch.uint8, device=d)
    p = B.drk_reward_params_default()
    assert B.drk_reward(zb, z, z, None, 8, p, z, None) == B.DRK_OK          # PR not needed by default
    p.prs_mode = B.DRK_PRS_SOFT
    assert B.drk_reward(zb, z, z, None, 8, p, z, zb, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_reward(zb, z, z, z, 8, p, z, None, check=False) == B.DRK_ERR_INVALID_ARG
    p.prs_mode = 5
    assert B.drk_reward(zb, z, z, z, 8, p, z, zb, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_reward(zb, z, z, z, 0, None, z, zb) == B.DRK_OK and B.drk_last_launch_count() == 0
