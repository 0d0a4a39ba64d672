"""drk_pg_logprob_fwd_noalloc: the forward log-prob call whose scratch is a fixed array inside the library,
for callers that cannot allocate device memory at call time (a framework that owns all of HBM through its
own pool, or a section that must avoid cudaMalloc's implicit synchronisation).

Checked against the ordinary entry point, which takes a caller-allocated workspace, on two calls in a row
with different inputs: the second call finds the first call's leftovers in the shared array and must not be
affected by them.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2602_05885_b200 import binding as B
from benchlib import synth
from tests.helpers import TOL_LOGP_BF16, TOL_LOGP_F32

pytestmark = pytest.mark.gpu


def _inputs(T, H, V, dtype, seed, dev):
    hidden, W, _ = synth.dense_operands(T, H, V, dtype, seed, "cpu")
    ids = synth.uniform_ids(T, V, seed + 1)
    return hidden.to(dev), W.to(dev), ids.to(dev)


def _both(hidden, W, ids, engine=B.DRK_ENGINE_AUTO):
    T, H = hidden.shape
    V = W.shape[0]
    dev = hidden.device
    code = B.DRK_BF16 if hidden.dtype == torch.bfloat16 else B.DRK_F32
    ref_logp, ref_lse, ref_status = B.pg_logprob_fwd(hidden, W, ids, engine)       # caller-allocated workspace
    logp = torch.full((T,), float("nan"), device=dev)
    lse = torch.full((T,), float("nan"), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.drk_pg_logprob_fwd_noalloc(hidden, W, code, ids, T, H, V, engine, logp, lse, status)
    assert B.drk_last_launch_count() == 2
    torch.cuda.synchronize()
    return (logp.cpu(), lse.cpu(), int(status.item())), (ref_logp.cpu(), ref_lse.cpu(), int(ref_status.item()))


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA, B.DRK_ENGINE_SIMT],
                         ids=["pairs", "single-cta", "ffma"])
@pytest.mark.parametrize("dtype,tol", [(torch.bfloat16, TOL_LOGP_BF16), (torch.float32, TOL_LOGP_F32)])
def test_two_calls_in_a_row_match_the_workspace_entry_point(dtype, tol, engine):
    # every route into the fixed array: CTA pairs, one CTA per tile, and the FFMA kernels (which fp32 inputs
    # always take, whatever the engine says)
    dev = torch.device("cuda:0")
    # first call: larger problem, with two invalid ids so that stale target logits would show up later
    h1, W1, ids1 = _inputs(700, 512, 9000, dtype, 21, dev)
    ids1[3] = -1
    ids1[650] = 9000
    got, ref = _both(h1, W1, ids1, engine)
    assert got[2] == ref[2] and (got[2] & B.DRK_STATUS_BAD_ID)
    assert (got[0] - ref[0]).abs().max() <= tol and (got[1] - ref[1]).abs().max() <= tol
    # second call, different sizes and data, right after the first
    h2, W2, ids2 = _inputs(333, 256, 4100, dtype, 22, dev)
    ids2[3] = 4100                                   # invalid again: its target must read as 0, not as a leftover
    got, ref = _both(h2, W2, ids2, engine)
    assert got[2] == ref[2]
    assert (got[0] - ref[0]).abs().max() <= tol and (got[1] - ref[1]).abs().max() <= tol
    assert abs(float(got[0][3]) + float(got[1][3])) < 1e-6
    assert torch.isfinite(got[0]).all() and torch.isfinite(got[1]).all()


def test_sizes_beyond_the_fixed_scratch_are_rejected():
    dev = torch.device("cuda:0")
    H, V = 64, 1 << 20                               # many vocabulary ranges per row: scratch per row is large
    T = 4000000
    z = torch.zeros(16, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    # rejected on the host before any pointer is touched
    rc = B.drk_pg_logprob_fwd_noalloc(z, z, B.DRK_BF16, z, T, H, V, 0, z, z, st, check=False)
    assert rc == B.DRK_ERR_WORKSPACE
    assert B.drk_last_launch_count() == 0
    assert "workspace" in B.drk_status_string(rc)
    # (the 14B training shape, T = 32768, needs about 2.2 MB of the fixed array: this entry point uses few,
    # long vocabulary ranges per row tile, unlike the workspace entry point)
