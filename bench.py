#!/usr/bin/env python
"""Throughput of the fused policy-gradient loss (TRLOO + MRS + LM-head fwd/bwd) on synthetic batches.

    python bench.py --gpus 1 --steps 10 --warmup 3
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference ...     # times the fp64 CPU oracle on a bounded sample

One step = one pass of the whole path over one packed micro-batch: drk_trloo_advantage over the rollout
batch, drk_segment_advantages (the per-sample advantages of the packed segments), drk_pg_loss_fwd_bwd.
Prints one JSON line.

--parallelism vocab (not the default) splits W by rows over the ranks instead of giving every rank its own
micro-batch: drk_pg_shard_stats_fwd, all-gather of the per-row statistics, drk_pg_shard_loss_bwd, all-reduce
of dH; the same micro-batch on every rank, so the scaling is strong.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fused PG-loss fwd+bwd tokens/s at H=5120,V=151936 bf16; % of dense BF16 peak"
UNIT = "tokens/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(tflops=float(d["bf16_tflops_sustained"]), burst=float(d["bf16_tflops"]),
                    hbm=float(d["hbm_gbs"]), source="measured")
    return dict(tflops=1400.0, burst=1590.0, hbm=6650.0, source="fallback")


KERNEL_SOURCES = ["umma_kernels.cu", "umma.cuh", "umma_plan.cuh", "compact.cu", "api.cu", "common.cuh"]
TRAFFIC_PROFILE = os.path.join(ROOT, "profiles", "umma_gemm_kernel_dram_traffic_model.md")


def kernel_source_hash() -> str:
    """sha256 over the sources that decide the tensor-core kernels' memory traffic (kernels, launch geometry)."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2602_05885_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def traffic_model(config: dict, rows_fwd: int, rows_bwd: int, n_chunks: int):
    """DRAM bytes (read + write) of one fused call, from the tracked ncu summary.

    The summary holds, per kernel instantiation, bytes = A + B * rows fitted to one-pass captures of
    dram__bytes_read.sum + dram__bytes_write.sum at two reduced row counts (same H, V and chunk width as the
    benchmark), together with the hash of the kernel sources and the configuration they were taken with.
    Returns (bytes, note); bytes is None when the sources or the configuration differ from the capture's."""
    import re
    if not os.path.exists(TRAFFIC_PROFILE):
        return None, "no tracked capture"
    text = open(TRAFFIC_PROFILE).read()
    m = re.search(r"```json\s*(\{.*?\})\s*```", text, flags=re.S)
    if not m:
        return None, "no model in the tracked capture"
    model = json.loads(m.group(1))
    if model.get("kernel_source_sha256") != kernel_source_hash():
        return None, "kernel sources changed since the capture"
    if any(model["config"].get(k) != v for k, v in config.items()) or model["config"].get("chunks") != n_chunks:
        return None, "configuration differs from the capture's"
    total = 0.0
    for mode, rows in (("FWD", rows_fwd), ("DL", rows_bwd), ("DW", rows_bwd), ("DH", rows_bwd)):
        total += model["bytes"][mode]["A"] + model["bytes"][mode]["B_per_row"] * rows
    return total, (f"A + B*rows per kernel, fitted to one-pass ncu captures at {model['fit_rows']} rows "
                   f"(checked at {model['check_rows']}: {model['check_error_pct']} % off), "
                   f"profiles/{os.path.basename(TRAFFIC_PROFILE)}")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons))


def run_reference(args):
    """Times the oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from oracle import drk_oracle as O
    from benchlib import workload
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    n_tok = args.ref_tokens
    wl = workload.build("qwen3-14b", "cpu", seed=2000, T_override=n_tok)
    hidden = wl.hidden.double().numpy()
    W = wl.W.double().numpy()
    ids = wl.ids.numpy()
    rl = wl.rollout_logp.double().numpy()
    mask = wl.loss_mask.numpy()
    cu = wl.cu.numpy()
    adv = np.ones(wl.S)

    def step():
        # the benchmark's default: acceptance band open, veto off (every sample retained)
        G = O.returns(wl.reward.numpy(), wl.valid.numpy(), 1.0)
        O.trloo_advantage(G, wl.valid.numpy(), wl.prompt_of_rollout.numpy())
        return O.pg_loss_fwd_bwd(hidden, W, ids, rl, mask, cu, adv, lo=0.0, hi=float("inf"), veto=0.0)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    val = n_tok * args.steps / dt
    sample = f"{n_tok} packed tokens per step at full H=5120, V=151936 (fp64 oracle: TRLOO + fwd + MRS + loss + dH + dW)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "qwen3-14b-shaped micro-batch, H=5120, V=151936", "sample_tokens": n_tok},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(n_tok: int):
    """The oracle timed once on a bounded sample of the same workload (host cores of this machine)."""
    import numpy as np
    from oracle import drk_oracle as O
    from benchlib import workload
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    wl = workload.build("qwen3-14b", "cpu", seed=2000, T_override=n_tok)
    hidden = wl.hidden.double().numpy()
    W = wl.W.double().numpy()
    t0 = time.perf_counter()
    G = O.returns(wl.reward.numpy(), wl.valid.numpy(), 1.0)
    O.trloo_advantage(G, wl.valid.numpy(), wl.prompt_of_rollout.numpy())
    O.pg_loss_fwd_bwd(hidden, W, wl.ids.numpy(), wl.rollout_logp.double().numpy(), wl.loss_mask.numpy(),
                      wl.cu.numpy(), np.ones(wl.S), lo=0.0, hi=float("inf"), veto=0.0)
    dt = time.perf_counter() - t0
    return {"value": n_tok / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"one pass over {n_tok} packed tokens at full H=5120, V=151936 in {dt:.1f} s "
                      "(fp64: TRLOO + full logits + log-softmax + MRS + loss + dH + dW)"}


def run_sweep(args):
    """Roofline sweep: T x V x H grid, bf16, equal-length segments, uniform ids.  One JSON line per point."""
    from paper_2602_05885_b200 import binding as B
    from benchlib import workload
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = measured_peaks()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    idx = 0
    for H in (4096, 5120):
        for V in (32768, 151936):
            for T in (4096, 8192, 16384, 32768, 65536):
                wl = workload.build("sweep", dev, seed=4000 + idx, sweep_shape=(T, V, H))
                idx += 1
                S = wl.S
                g = torch.Generator(device=dev).manual_seed(idx)
                seg_adv = torch.randn(S, generator=g, device=dev)
                row = {"sweep_point": {"T": T, "V": V, "H": H}, "unit": UNIT}
                for mode in ("wide", "off"):
                    p = B.drk_pg_params_default()
                    if mode == "wide":
                        p.mrs_lo, p.mrs_hi = wl.wide_band()
                    else:
                        p.mrs_lo, p.mrs_hi, p.veto_ratio = 0.0, float("inf"), 0.0
                    p.dh_dtype = B.DRK_BF16
                    bufs = B.PgLossBuffers(T, H, V, S, B.DRK_BF16, p, dev)

                    def call():
                        B.drk_pg_loss_fwd_bwd(wl.hidden, wl.W, B.DRK_BF16, wl.ids, wl.rollout_logp, wl.loss_mask, wl.cu,
                                              seg_adv, T, H, V, S, p, bufs.loss, bufs.logp, bufs.lse, None, bufs.seg_w,
                                              bufs.seg_keep, bufs.counters, bufs.dH, bufs.dW, bufs.workspace,
                                              bufs.workspace_bytes, bufs.status)
                    for _ in range(3):
                        call()
                    torch.cuda.synchronize()
                    e0.record()
                    for _ in range(args.steps):
                        call()
                    e1.record()
                    torch.cuda.synchronize()
                    ms = e0.elapsed_time(e1) / args.steps
                    Tc = int(bufs.counters[0].item())     # advantages are non-zero here: kept tokens = backward rows
                    tf = (2.0 * T + 6.0 * Tc) * H * V / (ms * 1e-3) / 1e12
                    row[mode] = {"ms": ms, "tokens_per_s": T / (ms * 1e-3), "rows_in_backward": Tc, "tflops": tf,
                                 "frac_of_measured_sustained": tf / peaks["tflops"], "frac_of_nominal_2250": tf / 2250.0,
                                 "status": int(bufs.status.item())}
                    del bufs
                print(json.dumps(row), flush=True)
                del wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3-14b", choices=["qwen3-14b", "qwen3-8b", "ragged", "tiny"])
    ap.add_argument("--tokens", type=int, default=0, help="override the micro-batch size T (smaller captures)")
    ap.add_argument("--dw-dtype", default="f32", choices=["f32", "bf16"])
    ap.add_argument("--dh-dtype", default="bf16", choices=["f32", "bf16"])
    ap.add_argument("--v-chunk", type=int, default=0)
    ap.add_argument("--forward-rows", default="all", choices=["all", "usable"],
                    help="usable: the forward skips rows that are not loss-masked tokens of a segment")
    ap.add_argument("--dw-exchange", default="all-reduce", choices=["all-reduce", "reduce-scatter"],
                    help="with --sync-dw: all-reduce every finished slice of dW, or reduce-scatter it so that each rank "
                         "keeps its 1/N of the rows (half the bytes; what a sharded optimizer needs)")
    ap.add_argument("--sync-dw", action="store_true",
                    help="all-reduce dW across ranks slice by slice as the backward finishes each vocabulary chunk "
                         "(overlapped on a second stream); off by default: the loss path itself needs no collective")
    ap.add_argument("--engine", default="auto", choices=["auto", "1cta"],
                    help="auto: tcgen05 kernels on CTA pairs; 1cta: one CTA per tile")
    ap.add_argument("--mrs", default="off", choices=["off", "wide", "paper"],
                    help="off (default): the acceptance band is open and the veto disabled, so every loss-masked token "
                         "goes through the backward (the full 8 T H V of work; the rejection kernels still run); "
                         "wide: a band that retains about half of the samples; paper: [0.999, 1.001] and the 1e-4 veto, "
                         "under which this workload's noise level rejects nearly every sample")
    ap.add_argument("--parallelism", default="data", choices=["data", "vocab"],
                    help="data: one micro-batch per rank, no collective on the loss path (weak scaling); "
                         "vocab: W split by rows over the ranks, one micro-batch for all (strong scaling)")
    ap.add_argument("--ref-tokens", type=int, default=256)
    ap.add_argument("--cpu-tokens", type=int, default=512)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="roofline sweep over T x V x H instead of the headline run")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return
    if args.sweep:
        run_sweep(args)
        return

    from paper_2602_05885_b200 import binding as B
    from paper_2602_05885_b200 import dp
    from benchlib import workload
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.load()

    # data parallel: every rank owns a different micro-batch of the same rollout batch (weak scaling);
    # vocabulary parallel: every rank sees the same micro-batch and owns a block of W's rows (strong scaling)
    vocab = args.parallelism == "vocab"
    wl = workload.build(args.workload, dev, seed=2000, microbatch=0 if vocab else rank,
                        T_override=args.tokens or None)
    T, H, V_total, S = wl.T, wl.H, wl.V, wl.S
    v_begin, v_end = dp.vocab_shards(V_total, world)[rank] if vocab else (0, V_total)
    if v_end <= v_begin:
        raise SystemExit("more ranks than vocabulary tiles")
    W_local = wl.W[v_begin:v_end].contiguous() if vocab else wl.W
    if vocab:
        wl.W = None
    V = v_end - v_begin
    code = B.DRK_F32 if wl.dtype == torch.float32 else B.DRK_BF16
    p = B.drk_pg_params_default()
    if args.mrs == "wide":
        p.mrs_lo, p.mrs_hi = wl.wide_band()
    elif args.mrs == "off":
        p.mrs_lo, p.mrs_hi, p.veto_ratio = 0.0, float("inf"), 0.0
    p.dw_dtype = B.DRK_BF16 if args.dw_dtype == "bf16" else B.DRK_F32
    p.dh_dtype = B.DRK_BF16 if args.dh_dtype == "bf16" else B.DRK_F32
    # vocabulary parallel on several ranks: every rank's dH is a partial sum, and the parts cross the ranks in
    # fp32; the requested bf16 is produced after the reduction
    dh_bf16_after = vocab and world > 1 and p.dh_dtype == B.DRK_BF16
    if dh_bf16_after:
        p.dh_dtype = B.DRK_F32
    p.v_chunk = args.v_chunk
    p.engine = B.DRK_ENGINE_UMMA_1CTA if args.engine == "1cta" else B.DRK_ENGINE_AUTO
    p.forward_rows = 1 if args.forward_rows == "usable" else 0
    bufs = B.PgLossBuffers(T, H, V, S, code, p, dev)
    R, Tmax = wl.reward.shape
    ret = torch.empty_like(wl.reward)
    adv = torch.empty_like(wl.reward)
    gsize = torch.empty((R, Tmax), dtype=torch.int32, device=dev)
    seg_rollout = wl.seg_rollout.to(torch.int32).contiguous()
    seg_turn = wl.seg_turn.to(torch.int32).contiguous()
    seg_adv = torch.empty(S, dtype=torch.float32, device=dev)
    stats = torch.empty((T, 4), dtype=torch.float32, device=dev)
    dh_out = torch.empty((T, H), dtype=torch.bfloat16, device=dev) if dh_bf16_after else None
    stream = torch.cuda.current_stream()
    launches = [0]
    comm = None
    if args.sync_dw and vocab:
        raise SystemExit("--sync-dw belongs to data parallelism: with W split by rows every rank owns its rows of dW")
    if args.sync_dw:
        # one event per vocabulary chunk; the communication stream reduces a slice of dW once its event fired
        n_chunks, vc = B.drk_pg_bwd_chunks(T, H, V, code, p)
        events = [torch.cuda.Event() for _ in range(n_chunks)]
        for e in events:
            e.record(stream)
        B.set_dw_chunk_events(p, [e.cuda_event for e in events])
        comm = torch.cuda.Stream()
        dw_shard = None
        if args.dw_exchange == "reduce-scatter":
            owned = dp.dw_shard_rows(V, vc, world, rank)
            dw_shard = torch.empty((sum(b - a for a, b in owned), H), dtype=bufs.dW.dtype, device=dev)

    def step(hidden, ids, rl, mask, cu, out=None):
        o = out if out is not None else bufs
        B.drk_trloo_advantage(wl.reward, wl.valid, wl.prompt_of_rollout, R, Tmax, 1.0, B.DRK_BASELINE_TRLOO,
                              ret, adv, gsize, o.status, stream)
        launches[0] += B.drk_last_launch_count()
        B.drk_segment_advantages(adv, seg_rollout, seg_turn, R, Tmax, S, seg_adv, o.status, stream)
        launches[0] += B.drk_last_launch_count()
        if vocab:
            launches[0] += dp.vocab_parallel_loss_fwd_bwd(hidden, W_local, ids, rl, mask, cu, seg_adv, v_begin, V_total,
                                                          p, o, stats, stream, dh_out)
            return
        B.drk_pg_loss_fwd_bwd(hidden, W_local, code, ids, rl, mask, cu, seg_adv, T, H, V, S, p, o.loss, o.logp,
                              o.lse, o.entropy, o.seg_w, o.seg_keep, o.counters, o.dH, o.dW,
                              o.workspace, o.workspace_bytes, o.status, stream)
        launches[0] += B.drk_last_launch_count()
        if comm is not None:
            if dw_shard is not None:
                dp.reduce_scatter_dw_slices(bufs.dW, vc, dw_shard, events, comm)
            else:
                dp.all_reduce_dw_slices(bufs.dW, vc, events, comm)
            stream.wait_stream(comm)        # the step ends when the last slice has been exchanged

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------------------------------------------------------- device-resident timing
    for _ in range(args.warmup):
        step(wl.hidden, wl.ids, wl.rollout_logp, wl.loss_mask, wl.cu)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches[0] = 0
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        step(wl.hidden, wl.ids, wl.rollout_logp, wl.loss_mask, wl.cu)
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    n_launch = launches[0]
    status = int(bufs.status.item())
    counters = bufs.counters.tolist()
    ms_max = dp.max_over_ranks(ms, dev)
    value = (1 if vocab else world) * T * args.steps / (ms_max * 1e-3)

    # ---------------------------------------------------------------- the fused call alone (roofline)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fused_launches = [0]

    def time_fused(pp, reps):
        out = []
        for _ in range(reps):
            e0.record(stream)
            if vocab:      # this rank's two calls with the exchange between them
                fused_launches[0] = dp.vocab_parallel_loss_fwd_bwd(wl.hidden, W_local, wl.ids, wl.rollout_logp,
                                                                   wl.loss_mask, wl.cu, seg_adv, v_begin, V_total, pp,
                                                                   bufs, stats, stream, dh_out)
            else:
                B.drk_pg_loss_fwd_bwd(wl.hidden, W_local, code, wl.ids, wl.rollout_logp, wl.loss_mask, wl.cu, seg_adv,
                                      T, H, V, S, pp, bufs.loss, bufs.logp, bufs.lse, bufs.entropy, bufs.seg_w,
                                      bufs.seg_keep, bufs.counters, bufs.dH, bufs.dW, bufs.workspace,
                                      bufs.workspace_bytes, bufs.status, stream)
                fused_launches[0] = B.drk_last_launch_count()
            e1.record(stream)
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1))
        return statistics.mean(out)

    def backward_rows():
        # rows the backward GEMMs process: loss-masked tokens of retained samples with a non-zero advantage
        keep = bufs.seg_keep.bool() & (seg_adv != 0)
        cu = wl.cu.long()
        csum = torch.cat([torch.zeros(1, dtype=torch.long, device=dev), wl.loss_mask.long().cumsum(0)])
        per_seg = csum[cu[1:]] - csum[cu[:-1]]
        return int((per_seg * keep.long()).sum().item())

    fused_ms = time_fused(p, min(args.steps, 5))
    # merge + 3 MRS + 4 compaction kernels + the dH scatter are not GEMM launches (the FFMA path has neither
    # compaction nor scatter; the vocabulary-parallel form has one more merge)
    n_gemm_launches = fused_launches[0] - (9 if code == B.DRK_BF16 else 4) - (1 if vocab else 0)
    Tc = backward_rows() if code == B.DRK_BF16 else T
    Tf = int(bufs.counters[1].item()) if (p.forward_rows == 1 and code == B.DRK_BF16) else T   # rows the forward ran on
    flops = (2.0 * Tf + 6.0 * Tc) * H * V
    peaks = measured_peaks()
    achieved = flops / (fused_ms * 1e-3) / 1e12
    n_chunks, vc_used = B.drk_pg_bwd_chunks(T, H, V, code, p)
    traffic, traffic_note = traffic_model(dict(H=H, V=V_total, v_chunk=vc_used, dW=args.dw_dtype, dH=args.dh_dtype,
                                               engine=args.engine, parallelism=args.parallelism, dtype="bf16" if
                                               code == B.DRK_BF16 else "f32"), Tf, Tc, n_chunks)
    # the same call with a band that retains about half of the samples: rows of rejected samples skip the backward
    wide = None
    if args.mrs == "off":
        p_w = B.drk_pg_params_default()
        for f, _ in p._fields_:
            setattr(p_w, f, getattr(p, f))
        p_w.mrs_lo, p_w.mrs_hi = wl.wide_band()
        p_w.veto_ratio = B.drk_pg_params_default().veto_ratio
        w_ms = time_fused(p_w, min(args.steps, 5))
        Tc_w = backward_rows() if code == B.DRK_BF16 else T
        w_tflops = (2.0 * Tf + 6.0 * Tc_w) * H * V / (w_ms * 1e-3) / 1e12
        wide = {"call_ms": w_ms, "rows_in_backward": Tc_w, "tflops": w_tflops, "frac": w_tflops / peaks["tflops"],
                "tokens_per_s": T / (w_ms * 1e-3),
                "what": "same call, acceptance band exp(-+q) around 1 with q between the middle order statistics of the "
                        "samples' |mean log-ratio| (about half retained), veto 1e-4"}
        time_fused(p, 1)   # leave the outputs of the configured run in the buffers

    # ---------------------------------------------------------------- end to end with host buffers
    e2e = None
    if not args.no_e2e:
        host = [t.cpu().pin_memory() for t in (wl.hidden, wl.ids, wl.rollout_logp, wl.loss_mask, wl.cu)]
        devin = [torch.empty_like(t, device=dev) for t in host]
        h_loss = torch.empty(1, dtype=torch.float32).pin_memory()
        h_cnt = torch.empty(4, dtype=torch.int64).pin_memory()
        h_logp = torch.empty(T, dtype=torch.float32).pin_memory()
        h_keep = torch.empty(S, dtype=torch.uint8).pin_memory()
        h_dH = torch.empty((T, H), dtype=bufs.dH.dtype).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in host)
        d2h = sum(t.numel() * t.element_size() for t in (h_loss, h_cnt, h_logp, h_keep, h_dH))

        # Two sets of device inputs and outputs: the upload of step i+1 and the download of step i-1 run on
        # their own streams while step i computes, as a trainer's input pipeline would do.  Every step still
        # moves its own inputs in and its own results out inside the timed region.
        bufs2 = B.PgLossBuffers(T, H, V, S, code, p, dev, dW=bufs.dW)
        out_sets = [bufs, bufs2]
        in_sets = [devin, [torch.empty_like(t, device=dev) for t in host]]
        up, down = torch.cuda.Stream(), torch.cuda.Stream()
        ev_up = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_down = [torch.cuda.Event() for _ in range(2)]

        def upload(k):
            with torch.cuda.stream(up):
                up.wait_event(ev_done[k])                 # the step that last read this input set has finished
                for src, dst in zip(host, in_sets[k]):
                    dst.copy_(src, non_blocking=True)
                ev_up[k].record(up)

        def download(k):
            with torch.cuda.stream(down):
                down.wait_event(ev_done[k])
                o = out_sets[k]
                h_loss.copy_(o.loss, non_blocking=True)
                h_cnt.copy_(o.counters, non_blocking=True)
                h_logp.copy_(o.logp, non_blocking=True)
                h_keep.copy_(o.seg_keep, non_blocking=True)
                h_dH.copy_(o.dH, non_blocking=True)
                ev_down[k].record(down)

        def e2e_run(n):
            for k in range(2):
                ev_done[k].record(stream)
                ev_down[k].record(stream)
            upload(0)
            for i in range(n):
                k = i % 2
                stream.wait_event(ev_up[k])               # this step's inputs have arrived
                stream.wait_event(ev_down[k])             # this output set has been read back (two steps ago)
                step(*in_sets[k], out=out_sets[k])
                ev_done[k].record(stream)
                if i + 1 < n:
                    upload(1 - k)
                download(k)
            stream.wait_stream(down)

        e2e_run(2)
        barrier()
        ev0.record(stream)
        e2e_run(args.steps)
        ev1.record(stream)
        barrier()
        e_ms = dp.max_over_ranks(ev0.elapsed_time(ev1), dev)
        e2e = {"value": (1 if vocab else world) * T * args.steps / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e_ms / args.steps,
               "what": "every step: hidden, ids, rollout log-probs, mask, cu_seqlens copied from pinned host memory; "
                       "loss, counters, log-probs, keep flags and dH copied back to pinned host memory; uploads and "
                       "downloads run on their own streams, double-buffered against the compute; W and dW stay "
                       "resident"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(args.cpu_tokens)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_max / args.steps, "higher_is_better": True,
            "scaling": "strong" if vocab else "weak",
            "vs_baseline": None, "dtype": "bf16" if code == B.DRK_BF16 else "f32", "data": "synthetic",
            "config": {"workload": f"{wl.name}-shaped packed micro-batch", "T": T, "H": H, "V": V_total, "V_local": V, "segments": S,
                       "rollout_batch": f"{R} rollouts x {Tmax} turns",
                       "mrs": {"off": "band open, veto off: every loss-masked token goes through the backward (8 T H V)",
                               "wide": "band retaining about half of the samples", "paper": "[0.999, 1.001], veto 1e-4"}[args.mrs],
                       "dW": args.dw_dtype, "dH": args.dh_dtype, "v_chunk": args.v_chunk or "default",
                       "engine": args.engine, "forward_rows": args.forward_rows,
                       "l2": "inputs exceed L2 (W alone is %.2f GB); no flush" % (V * H * 2 / 1e9),
                       "parallelism": (f"vp{world}: W split by rows ({V} of {V_total} on rank 0), one micro-batch for "
                                       "all ranks; all-gather of per-row statistics, all-reduce of dH") if vocab else
                                      (f"dp{world}: one micro-batch per rank, " +
                                       (f"dW exchanged per vocabulary chunk ({args.dw_exchange}), overlapped" if args.sync_dw
                                        else "no collective on the loss path"))},
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peaks["tflops"], "unit": "TFLOP/s",
                         "frac": achieved / peaks["tflops"], "traffic": traffic, "traffic_source": traffic_note,
                         "kernel": "umma_gemm_kernel (all four instantiations inside one drk_pg_loss_fwd_bwd call)",
                         "flops_per_call": flops, "call_ms": fused_ms, "gemm_launches_per_call": n_gemm_launches,
                         "flops_rule": "(2 T + 6 Tc) H V: forward over all T rows, backward over the Tc rows with "
                                       "a non-zero coefficient (rows of rejected or masked tokens are skipped)",
                         "rows_in_backward": Tc, "rows_in_forward": Tf,
                         "peak_source": f"bf16_tflops_sustained of {peaks['source']}",
                         "frac_of_burst": achieved / peaks["burst"], "frac_of_nominal_2250": achieved / 2250.0,
                         # the chip's dense bf16 rate at the clock it actually ran at (nominal 2250 TFLOP/s at the
                         # maximum SM clock, scaled by the median clock sampled during the timed region)
                         "frac_of_nominal_at_sampled_clock": (achieved / (2250.0 * clocks["sm_mhz"] / clocks["sm_max_mhz"])
                                                              if clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz")
                                                              else None)},
            "with_rejection_wide_band": wide,
            "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": n_launch, "clocks": clocks,
            "status_word": status, "counters": {"kept_tokens": counters[0], "masked_tokens": counters[1],
                                                "kept_segments": counters[2], "vetoed_segments": counters[3]},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
