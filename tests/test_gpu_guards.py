"""Out-of-bounds writes: every output buffer and the workspace sit between guard regions filled with a
byte pattern; after the call the guards must be untouched and the workspace must not have been written
beyond the size the library asked for.  Sizes are ragged in every dimension (row tiles, vocabulary tiles,
k-blocks and vocabulary chunks all end in partial ones)."""
import math

import pytest
import torch

from paper_2602_05885_b200 import binding as B
from tests import helpers as Hh
from tests.gpu_utils import make_params

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5


class GuardedArena:
    """Carves tensors out of one device byte buffer, each with GUARD bytes of PATTERN on both sides."""

    def __init__(self, device, nbytes):
        self.buf = torch.full((nbytes,), PATTERN, dtype=torch.uint8, device=device)
        self.off = 0
        self.guards = []

    def take(self, shape, dtype):
        n = int(math.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        start = (self.off + GUARD + 255) // 256 * 256
        self.guards.append((self.off, start))
        end = start + n
        self.off = (end + 255) // 256 * 256
        assert self.off + GUARD <= self.buf.numel(), "arena too small"
        view = self.buf[start:end].view(dtype).view(*shape) if n > 0 else torch.empty(shape, dtype=dtype, device=self.buf.device)
        self.guards.append((end, self.off))
        return view

    def check(self):
        torch.cuda.synchronize()
        spans = self.guards + [(self.off, min(self.off + GUARD, self.buf.numel()))]
        for a, b in spans:
            if b > a:
                assert bool((self.buf[a:b] == PATTERN).all()), f"guard bytes [{a},{b}) were overwritten"


def _guarded_buffers(case, p, dev):
    T, H, V, S = case.T, case.H, case.V, case.S
    code = B.DRK_F32 if case.dtype == torch.float32 else B.DRK_BF16
    nws = B.drk_pg_workspace_bytes(T, H, V, S, code, p, 1)
    dh_t = torch.bfloat16 if p.dh_dtype == B.DRK_BF16 else torch.float32
    dw_t = torch.bfloat16 if p.dw_dtype == B.DRK_BF16 else torch.float32
    total = nws + 4 * T * H + 4 * V * H + 64 * T + 64 * S + 64 * GUARD
    arena = GuardedArena(dev, total)
    bufs = B.PgLossBuffers.__new__(B.PgLossBuffers)
    bufs.loss = arena.take((1,), torch.float32)
    bufs.logp = arena.take((T,), torch.float32)
    bufs.lse = arena.take((T,), torch.float32)
    bufs.entropy = arena.take((T,), torch.float32)
    bufs.seg_w = arena.take((S,), torch.float32)
    bufs.seg_keep = arena.take((S,), torch.uint8)
    bufs.counters = arena.take((4,), torch.int64)
    bufs.dH = arena.take((T, H), dh_t)
    bufs.dW = arena.take((V, H), dw_t)
    bufs.status = arena.take((1,), torch.int32)
    bufs.status.zero_()
    bufs.workspace = arena.take((nws,), torch.uint8)
    bufs.workspace_bytes = nws
    return arena, bufs


@pytest.mark.parametrize("engine,dtype", [(B.DRK_ENGINE_AUTO, torch.bfloat16), (B.DRK_ENGINE_UMMA_1CTA, torch.bfloat16),
                                          (B.DRK_ENGINE_SIMT, torch.bfloat16), (B.DRK_ENGINE_AUTO, torch.float32)])
@pytest.mark.parametrize("T,H,V,vc", [(333, 264, 1100, 512), (700, 520, 2307, 0), (129, 72, 257, 256)])
@pytest.mark.parametrize("grad_dtype", [B.DRK_F32, B.DRK_BF16])
def test_fused_call_stays_inside_its_buffers(engine, dtype, T, H, V, vc, grad_dtype):
    dev = torch.device("cuda:0")
    case = Hh.build_plain_case("guard", T=T, H=H, V=V, dtype=dtype, S=5, seed=T + V, mask_frac=0.2)
    lo, hi = Hh.wide_band(case)
    for forward_rows in (0, 1):
        p = make_params(lo, hi, 1e-4, engine=engine, v_chunk=vc, dw_dtype=grad_dtype, dh_dtype=grad_dtype,
                        forward_rows=forward_rows)
        arena, bufs = _guarded_buffers(case, p, dev)
        for t in (bufs.dH, bufs.dW, bufs.logp, bufs.lse, bufs.entropy):
            t.fill_(float("nan"))                      # unwritten elements would show
        B.pg_loss_fwd_bwd(case.hidden.to(dev), case.W.to(dev), case.ids.to(dev), case.rollout_logp.to(dev),
                          case.loss_mask.to(dev), case.cu.to(dev), case.seg_adv.to(dev), p, bufs)
        arena.check()
        assert int(bufs.status.item()) == 0
        # the outputs themselves were fully written
        assert torch.isfinite(bufs.dH.float()).all() and torch.isfinite(bufs.dW.float()).all()
        if forward_rows == 0:
            err = (bufs.logp.double().cpu() - torch.from_numpy(case.logp)).abs().max()
            assert float(err) <= (Hh.TOL_LOGP_F32 if dtype == torch.float32 else Hh.TOL_LOGP_BF16)


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA, B.DRK_ENGINE_SIMT])
def test_forward_call_stays_inside_its_buffers(engine):
    dev = torch.device("cuda:0")
    T, H, V = 515, 136, 4099
    case = Hh.build_plain_case("guard-fwd", T=T, H=H, V=V, dtype=torch.bfloat16, S=3, seed=9)
    p = make_params(engine=engine)
    nws = B.drk_pg_workspace_bytes(T, H, V, 0, B.DRK_BF16, p, 0)
    arena = GuardedArena(dev, nws + 64 * T + 16 * GUARD)
    logp = arena.take((T,), torch.float32)
    lse = arena.take((T,), torch.float32)
    ent = arena.take((T,), torch.float32)
    status = arena.take((1,), torch.int32)
    status.zero_()
    ws = arena.take((nws,), torch.uint8)
    B.drk_pg_logprob_fwd(case.hidden.to(dev), case.W.to(dev), B.DRK_BF16, case.ids.to(dev), T, H, V, engine, logp, lse,
                         ent, ws, nws, status)
    arena.check()
    assert int(status.item()) == 0
    assert float((logp.double().cpu() - torch.from_numpy(case.logp)).abs().max()) <= Hh.TOL_LOGP_BF16


def test_advantage_call_stays_inside_its_buffers():
    dev = torch.device("cuda:0")
    R, Tmax = 37, 5
    g = torch.Generator().manual_seed(2)
    reward = torch.rand((R, Tmax), generator=g).to(dev)
    valid = (torch.rand((R, Tmax), generator=g) < 0.8).to(torch.uint8).to(dev)
    prompt = torch.sort(torch.randint(0, 6, (R,), generator=g)).values.to(torch.int32).to(dev)
    arena = GuardedArena(dev, 64 * R * Tmax + 16 * GUARD)
    ret = arena.take((R, Tmax), torch.float32)
    adv = arena.take((R, Tmax), torch.float32)
    gsize = arena.take((R, Tmax), torch.int32)
    B.drk_trloo_advantage(reward, valid, prompt, R, Tmax, 1.0, B.DRK_BASELINE_TRLOO, ret, adv, gsize)
    arena.check()
    assert torch.isfinite(adv).all() and int(gsize.max()) <= R
