"""ctypes binding of libdrk.so: argument marshalling only.

Every function has the name and argument order of its C entry point in
include/drk.h and takes torch tensors (device memory) where the C call takes
device pointers.  Nothing is computed here, and there is no fallback: if the
shared library is missing the import of a symbol raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

DRK_OK = 0
DRK_ERR_INVALID_ARG = -1
DRK_ERR_UNSUPPORTED = -2
DRK_ERR_WORKSPACE = -3
DRK_ERR_CUDA = -4
DRK_ERR_ARCH = -5

DRK_F32 = 0
DRK_BF16 = 1
DRK_BASELINE_TRLOO = 0
DRK_BASELINE_GRPO = 1
DRK_NORM_KEPT_TOKENS = 0
DRK_NORM_ALL_MASKED_TOKENS = 1
DRK_NORM_EXPLICIT = 2
DRK_ENGINE_AUTO = 0
DRK_ENGINE_SIMT = 1
DRK_ENGINE_UMMA_1CTA = 2

DRK_SCHEDULE_DYNAMIC = 0
DRK_SCHEDULE_STATIC = 1

DRK_STATUS_BAD_ID = 1
DRK_STATUS_BAD_SEGMENTS = 2
DRK_STATUS_NONFINITE = 4
DRK_STATUS_TIMEOUT = 8
DRK_STATUS_BAD_GROUPS = 16
DRK_STATUS_BOUNDS = 32


class drk_pg_params(ctypes.Structure):
    _fields_ = [
        ("mrs_lo", ctypes.c_float),
        ("mrs_hi", ctypes.c_float),
        ("veto_ratio", ctypes.c_float),
        ("norm", ctypes.c_int32),
        ("explicit_scale", ctypes.c_float),
        ("dw_dtype", ctypes.c_int32),
        ("dh_dtype", ctypes.c_int32),
        ("dw_accumulate", ctypes.c_int32),
        ("engine", ctypes.c_int32),
        ("v_chunk", ctypes.c_int32),
        ("keep_from_caller", ctypes.c_int32),
        ("forward_rows", ctypes.c_int32),
        ("dw_chunk_events", ctypes.POINTER(ctypes.c_void_p)),
        ("n_dw_chunk_events", ctypes.c_int32),
        ("reuse_forward", ctypes.c_int32),
        ("schedule", ctypes.c_int32),
    ]


class drk_reward_params(ctypes.Structure):
    _fields_ = [
        ("speedup_clip", ctypes.c_float),
        ("use_pr", ctypes.c_int32),
        ("prs_mode", ctypes.c_int32),
        ("prs_tau", ctypes.c_float),
        ("prs_s", ctypes.c_float),
        ("seed", ctypes.c_uint64),
        ("offset", ctypes.c_uint64),
    ]


DRK_PRS_OFF, DRK_PRS_SOFT, DRK_PRS_HARD = 0, 1, 2


class DrkError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


_lib: Optional[ctypes.CDLL] = None


def library_path() -> str:
    """The in-tree libdrk.so, or the build named by the environment variable DRK_LIBRARY (for instance the
    checked build libdrk_check.so, whose kernels range-check every index they derive on the device)."""
    return os.environ.get("DRK_LIBRARY") or _build.LIB_PATH


def load() -> ctypes.CDLL:
    """Loads libdrk.so (built in-tree by build.py).  Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it first (python -m paper_2602_05885_b200.build); "
            "there is no fallback path")
    lib = ctypes.CDLL(path)
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    lib.drk_pg_params_default.argtypes = [ctypes.POINTER(drk_pg_params)]
    lib.drk_pg_params_default.restype = None
    lib.drk_pg_bwd_chunks.argtypes = [i64, i32, i32, i32, ctypes.POINTER(drk_pg_params), ctypes.POINTER(ctypes.c_int32)]
    lib.drk_pg_bwd_chunks.restype = ctypes.c_int
    lib.drk_pg_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, ctypes.POINTER(drk_pg_params), i32]
    lib.drk_pg_workspace_bytes.restype = sz
    lib.drk_trloo_advantage.argtypes = [vp, vp, vp, i32, i32, f32, i32, vp, vp, vp, vp, vp]
    lib.drk_trloo_advantage.restype = ctypes.c_int
    lib.drk_pg_logprob_fwd.argtypes = [vp, vp, i32, vp, i64, i32, i32, i32, vp, vp, vp, vp, sz, vp, vp]
    lib.drk_pg_logprob_fwd.restype = ctypes.c_int
    lib.drk_reward_params_default.argtypes = [ctypes.POINTER(drk_reward_params)]
    lib.drk_reward_params_default.restype = None
    lib.drk_reward.argtypes = [vp, vp, vp, vp, i64, ctypes.POINTER(drk_reward_params), vp, vp, vp]
    lib.drk_reward.restype = ctypes.c_int
    lib.drk_pg_logprob_fwd_noalloc.argtypes = [vp, vp, i32, vp, i64, i32, i32, i32, vp, vp, vp, vp]
    lib.drk_pg_logprob_fwd_noalloc.restype = ctypes.c_int
    lib.drk_pg_loss_fwd_bwd.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, i64, i32, i32, i32,
                                        ctypes.POINTER(drk_pg_params), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz,
                                        vp, vp]
    lib.drk_pg_diagnostics.argtypes = [vp, vp, vp, vp, vp, i64, i32, vp, i32, vp, i32, i32, i32, vp, vp]
    lib.drk_pg_diagnostics.restype = ctypes.c_int
    lib.drk_pg_loss_fwd_bwd.restype = ctypes.c_int
    lib.drk_pg_shard_stats_fwd.argtypes = [vp, vp, i32, vp, i64, i32, i32, i32, i32, i32, vp, vp, sz, vp, vp]
    lib.drk_pg_shard_stats_fwd.restype = ctypes.c_int
    lib.drk_pg_shard_loss_bwd.argtypes = [vp, vp, i32, vp, vp, i32, vp, vp, vp, vp, i64, i32, i32, i32, i32, i32,
                                          ctypes.POINTER(drk_pg_params), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz,
                                          vp, vp]
    lib.drk_pg_shard_loss_bwd.restype = ctypes.c_int
    lib.drk_pg_shard_merge.argtypes = [vp, i32, vp, i64, i32, vp, vp, vp, vp, vp]
    lib.drk_pg_shard_merge.restype = ctypes.c_int
    lib.drk_segment_advantages.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp]
    lib.drk_segment_advantages.restype = ctypes.c_int
    lib.drk_selftest_bounded_wait.argtypes = [ctypes.c_uint32, vp, vp, vp]
    lib.drk_selftest_bounded_wait.restype = ctypes.c_int
    lib.drk_last_launch_count.argtypes = []
    lib.drk_last_launch_count.restype = ctypes.c_int
    lib.drk_selftest_fail_tensor_map.argtypes = [i32]
    lib.drk_selftest_fail_tensor_map.restype = None
    lib.drk_bounds_checked.argtypes = []
    lib.drk_bounds_checked.restype = ctypes.c_int
    lib.drk_tensor_map_encodes.argtypes = []
    lib.drk_tensor_map_encodes.restype = ctypes.c_uint64
    lib.drk_status_string.argtypes = [ctypes.c_int]
    lib.drk_status_string.restype = ctypes.c_char_p
    lib.drk_version.argtypes = []
    lib.drk_version.restype = ctypes.c_int
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("the C ABI takes dense row-major arrays: pass a contiguous tensor")
    return t.data_ptr() if t.numel() > 0 else (t.data_ptr() or None)


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DRK_F32
    if t.dtype == torch.bfloat16:
        return DRK_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def drk_status_string(code: int) -> str:
    return load().drk_status_string(int(code)).decode()


status_string = drk_status_string


def drk_version() -> int:
    return load().drk_version()


def drk_last_launch_count() -> int:
    return load().drk_last_launch_count()


def drk_selftest_fail_tensor_map(nth: int) -> None:
    load().drk_selftest_fail_tensor_map(int(nth))


def drk_bounds_checked() -> int:
    return int(load().drk_bounds_checked())


def drk_tensor_map_encodes() -> int:
    return int(load().drk_tensor_map_encodes())


def drk_pg_params_default() -> drk_pg_params:
    p = drk_pg_params()
    load().drk_pg_params_default(ctypes.byref(p))
    return p


def drk_pg_bwd_chunks(T: int, H: int, V: int, in_dtype: int, p: Optional[drk_pg_params]):
    """Returns (number of vocabulary chunks of the backward, chunk width)."""
    vc = ctypes.c_int32(0)
    n = load().drk_pg_bwd_chunks(T, H, V, in_dtype, ctypes.byref(p) if p is not None else None, ctypes.byref(vc))
    if n < 0:
        raise DrkError(n, "drk_pg_bwd_chunks")
    return n, int(vc.value)


def set_dw_chunk_events(p: drk_pg_params, handles) -> None:
    """Stores raw cudaEvent_t handles (ints) in p; the array is kept alive on p."""
    arr = (ctypes.c_void_p * len(handles))(*handles)
    p._dw_event_array = arr
    p.dw_chunk_events = ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p))
    p.n_dw_chunk_events = len(handles)


def drk_pg_workspace_bytes(T: int, H: int, V: int, S: int, in_dtype: int,
                           p: Optional[drk_pg_params], which: int) -> int:
    return int(load().drk_pg_workspace_bytes(T, H, V, S, in_dtype, ctypes.byref(p) if p is not None else None, which))


def drk_reward_params_default() -> drk_reward_params:
    p = drk_reward_params()
    load().drk_reward_params_default(ctypes.byref(p))
    return p


def drk_reward(correct, t_ref, t_kernel, pr, n: int, p: Optional[drk_reward_params], reward, retain, stream=None,
               check: bool = True) -> int:
    rc = load().drk_reward(_ptr(correct), _ptr(t_ref), _ptr(t_kernel), _ptr(pr), n,
                           ctypes.byref(p) if p is not None else None, _ptr(reward), _ptr(retain), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_reward")
    return rc


def drk_trloo_advantage(reward, valid, prompt_of_rollout, R: int, Tmax: int, gamma: float, baseline: int,
                        ret, adv, gsize, status=None, stream=None, check: bool = True) -> int:
    rc = load().drk_trloo_advantage(_ptr(reward), _ptr(valid), _ptr(prompt_of_rollout), R, Tmax, gamma, baseline,
                                    _ptr(ret), _ptr(adv), _ptr(gsize), _ptr(status), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_trloo_advantage")
    return rc


def drk_pg_logprob_fwd(hidden, W, in_dtype: int, ids, T: int, H: int, V: int, engine: int, logp, lse, entropy,
                       workspace, workspace_bytes: int, status, stream=None, check: bool = True) -> int:
    rc = load().drk_pg_logprob_fwd(_ptr(hidden), _ptr(W), in_dtype, _ptr(ids), T, H, V, engine, _ptr(logp), _ptr(lse),
                                   _ptr(entropy), _ptr(workspace), workspace_bytes, _ptr(status), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_pg_logprob_fwd")
    return rc


DRK_NOALLOC_SCRATCH_BYTES = 8 << 20


def drk_pg_logprob_fwd_noalloc(hidden, W, in_dtype: int, ids, T: int, H: int, V: int, engine: int, logp, lse,
                               status, stream=None, check: bool = True) -> int:
    """drk_pg_logprob_fwd without a workspace argument: the scratch is a fixed array inside libdrk.so
    (DRK_NOALLOC_SCRATCH_BYTES per GPU), for callers that cannot allocate device memory at call time.
    Sizes that need more return DRK_ERR_WORKSPACE.  Calls on one device share the array: keep them on one
    stream or otherwise ordered.  Make the first call on a device outside any stream capture."""
    rc = load().drk_pg_logprob_fwd_noalloc(_ptr(hidden), _ptr(W), in_dtype, _ptr(ids), T, H, V, engine, _ptr(logp),
                                           _ptr(lse), _ptr(status), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_pg_logprob_fwd_noalloc")
    return rc


def drk_pg_loss_fwd_bwd(hidden, W, in_dtype: int, ids, rollout_logp, loss_mask, cu_seqlens, seg_adv,
                        T: int, H: int, V: int, S: int, p: Optional[drk_pg_params], loss, logp, lse, entropy,
                        seg_w, seg_keep, counters, dH, dW, workspace, workspace_bytes: int, status, stream=None,
                        check: bool = True) -> int:
    rc = load().drk_pg_loss_fwd_bwd(_ptr(hidden), _ptr(W), in_dtype, _ptr(ids), _ptr(rollout_logp), _ptr(loss_mask),
                                    _ptr(cu_seqlens), _ptr(seg_adv), T, H, V, S,
                                    ctypes.byref(p) if p is not None else None, _ptr(loss), _ptr(logp), _ptr(lse),
                                    _ptr(entropy), _ptr(seg_w), _ptr(seg_keep), _ptr(counters), _ptr(dH), _ptr(dW),
                                    _ptr(workspace), workspace_bytes, _ptr(status), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_pg_loss_fwd_bwd")
    return rc


def drk_pg_shard_stats_fwd(hidden, W_shard, in_dtype: int, ids, T: int, H: int, V_local: int, v_begin: int,
                           V_total: int, engine: int, stats, workspace, workspace_bytes: int, status, stream=None,
                           check: bool = True) -> int:
    rc = load().drk_pg_shard_stats_fwd(_ptr(hidden), _ptr(W_shard), in_dtype, _ptr(ids), T, H, V_local, v_begin,
                                       V_total, engine, _ptr(stats), _ptr(workspace), workspace_bytes, _ptr(status),
                                       _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_pg_shard_stats_fwd")
    return rc


def drk_pg_shard_merge(stats_all, n_shards: int, ids, T: int, V_total: int, logp, lse, entropy, status, stream=None,
                       check: bool = True) -> int:
    rc = load().drk_pg_shard_merge(_ptr(stats_all), n_shards, _ptr(ids), T, V_total, _ptr(logp), _ptr(lse),
                                   _ptr(entropy), _ptr(status), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_pg_shard_merge")
    return rc


def drk_pg_shard_loss_bwd(hidden, W_shard, in_dtype: int, ids, stats_all, n_shards: int, rollout_logp, loss_mask,
                          cu_seqlens, seg_adv, T: int, H: int, V_local: int, v_begin: int, V_total: int, S: int,
                          p: Optional[drk_pg_params], loss, logp, lse, entropy, seg_w, seg_keep, counters, dH_part,
                          dW_shard, workspace, workspace_bytes: int, status, stream=None, check: bool = True) -> int:
    rc = load().drk_pg_shard_loss_bwd(_ptr(hidden), _ptr(W_shard), in_dtype, _ptr(ids), _ptr(stats_all), n_shards,
                                      _ptr(rollout_logp), _ptr(loss_mask), _ptr(cu_seqlens), _ptr(seg_adv), T, H,
                                      V_local, v_begin, V_total, S, ctypes.byref(p) if p is not None else None,
                                      _ptr(loss), _ptr(logp), _ptr(lse), _ptr(entropy), _ptr(seg_w), _ptr(seg_keep),
                                      _ptr(counters), _ptr(dH_part), _ptr(dW_shard), _ptr(workspace), workspace_bytes,
                                      _ptr(status), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_pg_shard_loss_bwd")
    return rc


def drk_segment_advantages(adv, seg_rollout, seg_turn, R: int, Tmax: int, S: int, seg_adv, status, stream=None,
                           check: bool = True) -> int:
    rc = load().drk_segment_advantages(_ptr(adv), _ptr(seg_rollout), _ptr(seg_turn), R, Tmax, S, _ptr(seg_adv),
                                       _ptr(status), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_segment_advantages")
    return rc


def drk_selftest_bounded_wait(limit_ms: int, status, waited_ns, stream=None, check: bool = True) -> int:
    rc = load().drk_selftest_bounded_wait(limit_ms, _ptr(status), _ptr(waited_ns), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_selftest_bounded_wait")
    return rc


def drk_pg_diagnostics(logp, rollout_logp, entropy, loss_mask, cu_seqlens, T: int, S: int, dH, dh_dtype: int,
                       dW, dw_dtype: int, H: int, V: int, out, stream=None, check: bool = True) -> int:
    rc = load().drk_pg_diagnostics(_ptr(logp), _ptr(rollout_logp), _ptr(entropy), _ptr(loss_mask), _ptr(cu_seqlens),
                                   T, S, _ptr(dH), dh_dtype, _ptr(dW), dw_dtype, H, V, _ptr(out), _stream(stream))
    if check and rc != DRK_OK:
        raise DrkError(rc, "drk_pg_diagnostics")
    return rc


DIAG_FIELDS = ("n_tokens", "mean_entropy", "ppl_train", "ppl_rollout", "mean_log_ratio", "max_abs_log_ratio",
               "grad_norm_dH", "grad_norm_dW")


# ---------------------------------------------------------------------------
# Convenience: allocate outputs and workspace with torch, then make the C call.
# ---------------------------------------------------------------------------

def _torch_dtype(code: int) -> torch.dtype:
    return torch.bfloat16 if code == DRK_BF16 else torch.float32


def trloo_advantage(reward: torch.Tensor, valid: torch.Tensor, prompt_of_rollout: torch.Tensor,
                    gamma: float = 1.0, baseline: int = DRK_BASELINE_TRLOO, status: Optional[torch.Tensor] = None):
    """Allocates ret/adv/gsize and calls drk_trloo_advantage.  Inputs are device tensors; `status` (device
    int32[1], optional) collects DRK_STATUS_BAD_GROUPS."""
    R, Tmax = reward.shape
    ret = torch.empty_like(reward)
    adv = torch.empty_like(reward)
    gsize = torch.empty((R, Tmax), dtype=torch.int32, device=reward.device)
    drk_trloo_advantage(reward.contiguous(), valid.contiguous(), prompt_of_rollout.contiguous(), R, Tmax,
                        gamma, baseline, ret, adv, gsize, status)
    return ret, adv, gsize


def pg_logprob_fwd(hidden: torch.Tensor, W: torch.Tensor, ids: torch.Tensor, engine: int = DRK_ENGINE_AUTO,
                   entropy: Optional[torch.Tensor] = None):
    T, H = hidden.shape
    V = W.shape[0]
    code = _dtype_code(hidden)
    p = drk_pg_params_default()
    p.engine = engine
    nbytes = drk_pg_workspace_bytes(T, H, V, 0, code, p, 0)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=hidden.device)
    logp = torch.empty(T, dtype=torch.float32, device=hidden.device)
    lse = torch.empty(T, dtype=torch.float32, device=hidden.device)
    status = torch.zeros(1, dtype=torch.int32, device=hidden.device)
    drk_pg_logprob_fwd(hidden, W, code, ids, T, H, V, engine, logp, lse, entropy, ws, nbytes, status)
    return logp, lse, status


class PgLossBuffers:
    """Outputs and workspace of drk_pg_loss_fwd_bwd for fixed sizes, allocated once."""

    def __init__(self, T: int, H: int, V: int, S: int, in_dtype: int, p: drk_pg_params, device,
                 dW: Optional[torch.Tensor] = None):
        self.T, self.H, self.V, self.S, self.in_dtype, self.p = T, H, V, S, in_dtype, p
        f32 = dict(dtype=torch.float32, device=device)
        self.loss = torch.zeros(1, **f32)
        self.logp = torch.empty(T, **f32)
        self.lse = torch.empty(T, **f32)
        self.entropy = torch.empty(T, **f32)
        self.seg_w = torch.empty(S, **f32)
        self.seg_keep = torch.empty(S, dtype=torch.uint8, device=device)
        self.counters = torch.zeros(4, dtype=torch.int64, device=device)
        self.dH = torch.empty((T, H), dtype=_torch_dtype(p.dh_dtype), device=device)
        self.dW = dW if dW is not None else torch.empty((V, H), dtype=_torch_dtype(p.dw_dtype), device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.workspace_bytes = drk_pg_workspace_bytes(T, H, V, S, in_dtype, p, 1)
        if self.workspace_bytes == 0:
            raise DrkError(DRK_ERR_INVALID_ARG, "drk_pg_workspace_bytes")
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=device)


def pg_loss_fwd_bwd(hidden, W, ids, rollout_logp, loss_mask, cu_seqlens, seg_adv,
                    p: Optional[drk_pg_params] = None, bufs: Optional[PgLossBuffers] = None, stream=None):
    T, H = hidden.shape
    V = W.shape[0]
    S = cu_seqlens.shape[0] - 1
    code = _dtype_code(hidden)
    if p is None:
        p = drk_pg_params_default()
    if bufs is None:
        bufs = PgLossBuffers(T, H, V, S, code, p, hidden.device)
    drk_pg_loss_fwd_bwd(hidden, W, code, ids, rollout_logp, loss_mask, cu_seqlens, seg_adv, T, H, V, S, p,
                        bufs.loss, bufs.logp, bufs.lse, bufs.entropy, bufs.seg_w, bufs.seg_keep, bufs.counters, bufs.dH,
                        bufs.dW,
                        bufs.workspace, bufs.workspace_bytes, bufs.status, stream)
    return bufs
