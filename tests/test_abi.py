"""The shared library loads without a GPU and exports what include/drk.h declares."""
import ctypes
import os
import re

import pytest
import torch

from paper_2602_05885_b200 import binding as B
from paper_2602_05885_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.load()


def _declared_functions():
    src = open(os.path.join(ROOT, "include", "drk.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(drk_[a-z0-9_]+)\s*\(", src)))


def test_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert {"drk_trloo_advantage", "drk_pg_logprob_fwd", "drk_pg_loss_fwd_bwd", "drk_pg_workspace_bytes",
            "drk_pg_params_default", "drk_status_string", "drk_version", "drk_last_launch_count"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    # and the binding offers a function of the same name for each
    for n in names:
        assert hasattr(B, n), n


def test_defaults_are_the_papers_constants():
    p = B.drk_pg_params_default()
    assert abs(p.mrs_lo - 0.999) < 1e-7 and abs(p.mrs_hi - 1.001) < 1e-7     # Sec. 5.1 acceptance band
    assert abs(p.veto_ratio - 1e-4) < 1e-10                                     # Sec. 5.1 token veto
    assert p.norm == B.DRK_NORM_KEPT_TOKENS and p.engine == B.DRK_ENGINE_AUTO
    assert ctypes.sizeof(B.drk_pg_params) == 72 and p.keep_from_caller == 0 and p.forward_rows == 0
    assert p.reuse_forward == 0 and p.schedule == B.DRK_SCHEDULE_DYNAMIC
    assert not p.dw_chunk_events and p.n_dw_chunk_events == 0


def test_workspace_bytes():
    p = B.drk_pg_params_default()
    small = B.drk_pg_workspace_bytes(1024, 256, 4096, 16, B.DRK_F32, p, 1)
    fwd = B.drk_pg_workspace_bytes(1024, 256, 4096, 16, B.DRK_F32, p, 0)
    assert 0 < fwd < small
    big = B.drk_pg_workspace_bytes(32768, 5120, 151936, 28, B.DRK_BF16, p, 1)
    # dL chunk (at most 2 GiB), gathered hidden rows, fp32 dH accumulator, per-row partials: a third of the bf16
    # logits (T x V), a sixth of the fp32 ones; a smaller v_chunk shrinks it further
    assert big < 0.35 * 32768 * 151936 * 2
    p.v_chunk = 7424
    assert B.drk_pg_workspace_bytes(32768, 5120, 151936, 28, B.DRK_BF16, p, 1) < 0.2 * 32768 * 151936 * 2
    p.v_chunk = 0
    # dH is accumulated in fp32 over the compacted rows whatever its own type: the workspace holds that buffer
    assert big >= 32768 * 5120 * 4
    p.dh_dtype = B.DRK_BF16
    assert B.drk_pg_workspace_bytes(32768, 5120, 151936, 28, B.DRK_BF16, p, 1) == big
    p.v_chunk = 16384
    assert B.drk_pg_workspace_bytes(32768, 5120, 151936, 28, B.DRK_BF16, p, 1) < big
    # invalid arguments give 0
    assert B.drk_pg_workspace_bytes(-1, 256, 4096, 16, B.DRK_F32, None, 1) == 0
    assert B.drk_pg_workspace_bytes(16, 256, 0, 16, B.DRK_F32, None, 1) == 0
    assert B.drk_pg_workspace_bytes(16, 256, 4096, 16, 5, None, 1) == 0
    assert B.drk_pg_workspace_bytes(16, 256, 4096, 16, B.DRK_F32, None, 2) == 0


def test_status_strings_and_version():
    assert B.drk_version() >= 100
    seen = {B.status_string(c) for c in range(0, -6, -1)}
    assert len(seen) == 6 and "unknown status" not in seen
    assert B.status_string(-99) == "unknown status"


def test_validation_precedes_any_cuda_call():
    # these are rejected on the host before the device is touched, so they behave the same without a GPU
    z = torch.zeros(8)
    assert B.drk_trloo_advantage(z, z, z, -1, 2, 1.0, 0, z, z, z, stream=0, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_trloo_advantage(z, z, z, 2, 2, 1.5, 0, z, z, z, stream=0, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_trloo_advantage(z, z, z, 2, 2, 1.0, 9, z, z, z, stream=0, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_trloo_advantage(z, z, z, 2, 65, 1.0, 0, z, z, z, stream=0, check=False) == B.DRK_ERR_UNSUPPORTED
    assert B.drk_trloo_advantage(None, z, z, 2, 2, 1.0, 0, z, z, z, stream=0, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_pg_logprob_fwd(z, z, B.DRK_BF16, z, 8, 0, 16, 0, z, z, None, z, 1 << 20, z, stream=0,
                                check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_last_launch_count() == 0


def test_validation_of_the_vocabulary_range_calls_and_the_gather():
    big = torch.zeros(256)
    off = (-big.data_ptr() % 256) // 4
    z = big[off:off + 64]                                    # 256-byte aligned, as a workspace must be
    p = B.drk_pg_params_default()
    fwd = lambda V_local, v_begin, V_total, T=8, H=8: B.drk_pg_shard_stats_fwd(
        z, z, B.DRK_BF16, z, T, H, V_local, v_begin, V_total, 0, z, z, 1 << 20, z, stream=0, check=False)
    assert fwd(16, 8, 16) == B.DRK_ERR_INVALID_ARG          # the range leaves the vocabulary
    assert fwd(16, -1, 64) == B.DRK_ERR_INVALID_ARG
    assert fwd(0, 0, 64) == B.DRK_ERR_INVALID_ARG
    assert fwd(16, 0, (1 << 24) + 1) == B.DRK_ERR_INVALID_ARG
    assert fwd(16, 0, 64, T=0) == B.DRK_OK                  # nothing to do, nothing enqueued
    bwd = lambda n_shards, v_begin, V_total, pp=p: B.drk_pg_shard_loss_bwd(
        z, z, B.DRK_BF16, z, z, n_shards, z, z, z, z, 8, 8, 16, v_begin, V_total, 1, pp, z, z, z, z, z, z, z, z, z, z,
        1 << 20, z, stream=0, check=False)
    assert bwd(0, 0, 64) == B.DRK_ERR_INVALID_ARG
    assert bwd(4097, 0, 64) == B.DRK_ERR_INVALID_ARG
    assert bwd(2, 56, 64) == B.DRK_ERR_INVALID_ARG
    p2 = B.drk_pg_params_default()
    p2.forward_rows = 1
    assert bwd(2, 0, 64, p2) == B.DRK_ERR_UNSUPPORTED        # no forward pass to restrict
    merge = lambda n, T, V: B.drk_pg_shard_merge(z, n, z, T, V, z, z, None, z, stream=0, check=False)
    assert merge(0, 8, 64) == B.DRK_ERR_INVALID_ARG and merge(2, -1, 64) == B.DRK_ERR_INVALID_ARG
    assert merge(2, 8, 0) == B.DRK_ERR_INVALID_ARG and merge(2, 0, 64) == B.DRK_OK
    assert B.drk_pg_shard_merge(None, 2, z, 8, 64, z, z, None, z, stream=0, check=False) == B.DRK_ERR_INVALID_ARG
    gather = lambda R, Tmax, S, a=z: B.drk_segment_advantages(a, z, z, R, Tmax, S, z, z, stream=0, check=False)
    assert gather(-1, 2, 4) == B.DRK_ERR_INVALID_ARG and gather(2, 2, -4) == B.DRK_ERR_INVALID_ARG
    assert gather(2, 2, 0) == B.DRK_OK
    assert gather(2, 2, 4, None) == B.DRK_ERR_INVALID_ARG
    st = torch.zeros(4)
    assert B.drk_selftest_bounded_wait(0, st, st, stream=0, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_selftest_bounded_wait(1001, st, st, stream=0, check=False) == B.DRK_ERR_INVALID_ARG
    assert B.drk_last_launch_count() == 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU behaviour")
def test_without_a_gpu_calls_fail_loudly():
    # well-formed arguments, but no device: an error code, never a CPU fallback
    z = torch.zeros(64)
    rc = B.drk_trloo_advantage(z, z, z, 2, 2, 1.0, 0, z, z, z, stream=0, check=False)
    assert rc in (B.DRK_ERR_CUDA, B.DRK_ERR_ARCH)
    with pytest.raises(B.DrkError):
        B.drk_trloo_advantage(z, z, z, 2, 2, 1.0, 0, z, z, z, stream=0)


def test_binding_rejects_strided_tensors():
    # the C ABI knows nothing of strides: a transposed or sliced-by-column tensor must not be passed silently
    z = torch.zeros((8, 8))
    with pytest.raises(ValueError):
        B.drk_trloo_advantage(z.t(), z, z, 2, 2, 1.0, 0, z, z, z, stream=0, check=False)
    with pytest.raises(ValueError):
        B.drk_segment_advantages(z[:, ::2], z, z, 2, 2, 1, z, z, stream=0, check=False)
