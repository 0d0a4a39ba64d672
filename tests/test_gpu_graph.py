"""The fused call makes no host synchronisation and no allocation, so a CUDA graph can hold it: capture
one call, replay it on new inputs copied into the captured buffers, and require the replayed results to
equal the directly launched ones bit for bit (both tensor-core engines and the FFMA engine)."""
import numpy as np
import pytest
import torch

from paper_2602_05885_b200 import binding as B
from tests import helpers as Hh
from tests.gpu_utils import make_params

pytestmark = pytest.mark.gpu

NAMES = ("loss", "logp", "lse", "entropy", "seg_w", "seg_keep", "counters", "dH", "dW", "status")


def _call(case_dev, p, bufs, stream=None):
    hidden, W, ids, rl, mask, cu, adv = case_dev
    B.pg_loss_fwd_bwd(hidden, W, ids, rl, mask, cu, adv, p, bufs, stream=stream)


@pytest.mark.parametrize("engine", [B.DRK_ENGINE_AUTO, B.DRK_ENGINE_UMMA_1CTA, B.DRK_ENGINE_SIMT])
def test_fused_call_replays_from_a_cuda_graph(engine):
    dev = torch.device("cuda:0")
    cases = [Hh.build_plain_case(f"graph{k}", T=900, H=264, V=2307, dtype=torch.bfloat16, S=6, seed=40 + k,
                                 mask_frac=0.3) for k in range(2)]
    lo, hi = Hh.wide_band(cases[0])
    p = make_params(lo, hi, float(np.float32(1e-4)), engine=engine, v_chunk=1024, dh_dtype=B.DRK_BF16)
    to_dev = lambda c: [t.to(dev) for t in (c.hidden, c.W, c.ids, c.rollout_logp, c.loss_mask, c.cu, c.seg_adv)]
    T, H, V, S = cases[0].T, cases[0].H, cases[0].V, cases[0].S

    # direct launches: the expected bits
    expected = []
    for c in cases:
        bufs = B.PgLossBuffers(T, H, V, S, B.DRK_BF16, p, dev)
        _call(to_dev(c), p, bufs)
        torch.cuda.synchronize()
        expected.append({n: getattr(bufs, n).clone() for n in NAMES})
        assert int(bufs.status.item()) == 0

    # capture one call on static buffers (the first call outside the capture has done the one-time set-up)
    static_in = to_dev(cases[0])
    bufs = B.PgLossBuffers(T, H, V, S, B.DRK_BF16, p, dev)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        _call(static_in, p, bufs, stream=side)                       # warm-up on the capture stream
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            _call(static_in, p, bufs, stream=torch.cuda.current_stream())
    torch.cuda.synchronize()

    for k in (1, 0, 1):
        for dst, src in zip(static_in, to_dev(cases[k])):
            dst.copy_(src)
        for n in ("dH", "dW", "logp"):
            getattr(bufs, n).fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        for n in NAMES:
            assert torch.equal(getattr(bufs, n), expected[k][n]), (k, n)
