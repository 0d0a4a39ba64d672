// C-ABI entry points of libdrk.so: argument validation, workspace carving, dispatch.
#include "common.cuh"
#include "umma_plan.cuh"
#include <cmath>
#include <limits>
#include <nvtx3/nvToolsExt.h>   // header-only; ranges cost nothing unless a profiler is attached

namespace drk {

thread_local int g_launches = 0;

int sm_count() {
  static int cached[64] = {};
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 148; }
  if (dev >= 0 && dev < 64 && cached[dev] > 0) return cached[dev];
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    return 148;
  }
  if (dev >= 0 && dev < 64) cached[dev] = n;
  return n;
}

namespace {

constexpr int kDefaultVChunk = 8192;

// Names a phase of the fused call on the profiler's timeline for as long as the object lives.
struct Range {
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
  Range(const Range&) = delete;
  Range& operator=(const Range&) = delete;
};

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_arch() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return DRK_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return DRK_ERR_CUDA;
  return major == 10 ? DRK_OK : DRK_ERR_ARCH;
}

bool use_simt(int in_dtype, int engine) { return in_dtype == DRK_F32 || engine == DRK_ENGINE_SIMT; }
int umma_ctas(int engine) { return engine == DRK_ENGINE_UMMA_1CTA ? 1 : 2; }
bool engine_ok(int e) { return e == DRK_ENGINE_AUTO || e == DRK_ENGINE_SIMT || e == DRK_ENGINE_UMMA_1CTA; }

bool sizes_ok(int64_t T, int H, int V, int in_dtype) {
  if (T < 0 || T > (1 << 24) || H < 1 || H > 65536 || V < 1 || V > (1 << 24)) return false;
  if (in_dtype != DRK_F32 && in_dtype != DRK_BF16) return false;
  return true;
}

// Chunk width for the tensor-core backward when the caller leaves it to the library: the multiple of
// 256 that minimises the modelled time of the three per-chunk kernels.  Each kernel is persistent
// over the device's SMs with 128x256 tiles, so its time is (waves of tiles) x (k-blocks per tile); a fixed
// cost per launch stands for fill and drain, and each chunk costs one more pass over the fp32 dH accumulator
// (T x H elements read and written through the memory-side add).  The dL buffer is kept below 2 GiB (a fifth of
// the bf16 logits at T=32768, V=151936): measured there, 30720-column chunks (5 chunks) are 2.5 % faster than
// 7424-column ones (21 chunks), 14848 (11 chunks) 1.2 %; callers short of memory pass a smaller v_chunk.
int auto_vchunk(int64_t T, int H, int V) {
  const int64_t sms = sm_count(), launch_cost = 96;
  const int64_t mt_T = ceil_div(T, 128), nt_H = ceil_div(H, 256), kb_H = ceil_div(H, 64), kb_T = ceil_div(T, 64);
  int64_t cap = ((int64_t)1 << 31) / (2 * (T > 0 ? T : 1)) / 256 * 256;
  if (cap < 8192) cap = 8192;
  if (cap > 32768) cap = 32768;
  const int64_t vmax = ceil_div(V, 256) * 256;
  // one accumulate pass over dH, in the model's unit (a 128x256x64 MMA block): T*H*8 bytes of traffic at about
  // the rate at which such a block's operands (48 KiB) stream in
  const double acc_pass = (double)T * (double)H * 8.0 / (48.0 * 1024.0) / (double)sms;
  int best = 0;
  double best_cost = 0;
  for (int64_t vc = 2048; vc <= cap; vc += 256) {
    double cost = 0;
    for (int64_t v0 = 0; v0 < V; v0 += vc) {
      const int64_t w = V - v0 < vc ? V - v0 : vc;
      cost += (double)(ceil_div(mt_T * ceil_div(w, 256), sms) * kb_H + launch_cost);   // DL
      cost += (double)(ceil_div(ceil_div(w, 128) * nt_H, sms) * kb_T + launch_cost);   // DW
      cost += (double)(ceil_div(mt_T * nt_H, sms) * ceil_div(w, 64) + launch_cost);    // DH
      cost += acc_pass;
    }
    if (best == 0 || cost < best_cost) { best = (int)vc; best_cost = cost; }
    if (vc >= vmax) break;
  }
  return best;
}

int round_vchunk(int v_chunk, int64_t T, int H, int V, bool simt) {
  int vc = v_chunk > 0 ? v_chunk : (simt ? kDefaultVChunk : auto_vchunk(T, H, V));
  vc = (int)(ceil_div(vc, 256) * 256);
  const int vmax = (int)(ceil_div(V, 256) * 256);
  return vc < vmax ? vc : vmax;
}

// Carves 256-byte aligned pieces off the caller's workspace.
struct Carver {
  char* base;
  size_t off = 0;
  explicit Carver(void* b) : base(static_cast<char*>(b)) {}
  void* take(size_t bytes) {
    void* p = base ? base + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  }
};

struct FwdWs {
  float* part;
  float* tgt;
  int nsplit;
  int32_t* sched;   // work counter of the forward kernel (tensor-core path)
};
FwdWs carve_fwd(Carver& c, int64_t T, int V, bool simt, int engine) {
  FwdWs w;
  w.nsplit = simt ? simt_nsplit(T, V) : umma_nsplit(T, V, umma_ctas(engine), false);
  w.part = static_cast<float*>(c.take(sizeof(float) * 4 * (size_t)w.nsplit * (size_t)T));
  w.tgt = static_cast<float*>(c.take(sizeof(float) * (size_t)T));
  w.sched = simt ? nullptr : static_cast<int32_t*>(c.take(sizeof(int32_t)));
  return w;
}

struct BwdWs {
  float* coeff;
  double* seg_stats;
  void* dL;
  float* dH_acc;
  int vc;
  // tensor-core path only: compaction of the rows with non-zero coefficient
  int32_t* blk_cnt;
  int32_t* blk_off;
  int32_t* n_rows;
  int32_t* rowmap;
  __nv_bfloat16* hidden_c;
  int32_t* sched;   // work counters of the backward kernels, three per vocabulary chunk
};
BwdWs carve_bwd(Carver& c, int64_t T, int H, int V, int S, bool simt, const drk_pg_params& p) {
  BwdWs w;
  w.vc = round_vchunk(p.v_chunk, T, H, V, simt);
  w.coeff = static_cast<float*>(c.take(sizeof(float) * (size_t)T));
  w.seg_stats = static_cast<double*>(c.take(sizeof(double) * 4 * (size_t)S));
  const size_t rows_cap = (size_t)(ceil_div(T, 256) * 256);   // dL also holds the zero rows that pad the last tile
  w.dL = c.take((simt ? 4 : 2) * (simt ? (size_t)T : rows_cap) * (size_t)w.vc);
  // tensor-core path: fp32 accumulator of dH over the compacted rows (whatever dH's own type); FFMA path: an
  // fp32 copy of dH only when dH itself is bf16
  if (!simt) w.dH_acc = static_cast<float*>(c.take(sizeof(float) * rows_cap * (size_t)H));
  else w.dH_acc = (p.dh_dtype == DRK_BF16) ? static_cast<float*>(c.take(sizeof(float) * (size_t)T * (size_t)H)) : nullptr;
  w.blk_cnt = w.blk_off = w.n_rows = w.rowmap = w.sched = nullptr;
  w.hidden_c = nullptr;
  if (!simt) {
    w.sched = static_cast<int32_t*>(c.take(sizeof(int32_t) * 3 * (size_t)ceil_div(V, w.vc)));
    const size_t nblk = (size_t)compact_blocks(T), len = (size_t)compact_map_len(T);
    w.blk_cnt = static_cast<int32_t*>(c.take(sizeof(int32_t) * nblk));
    w.blk_off = static_cast<int32_t*>(c.take(sizeof(int32_t) * nblk));
    w.n_rows = static_cast<int32_t*>(c.take(sizeof(int32_t) * 2));
    w.rowmap = static_cast<int32_t*>(c.take(sizeof(int32_t) * len));
    w.hidden_c = static_cast<__nv_bfloat16*>(c.take(2 * len * (size_t)H));
  }
  return w;
}

bool params_ok(const drk_pg_params& p) {
  if (p.norm < 0 || p.norm > 2) return false;
  if (p.dw_dtype != DRK_F32 && p.dw_dtype != DRK_BF16) return false;
  if (p.dh_dtype != DRK_F32 && p.dh_dtype != DRK_BF16) return false;
  if (!engine_ok(p.engine)) return false;
  if (p.v_chunk < 0) return false;
  if (p.keep_from_caller < 0 || p.keep_from_caller > 2) return false;
  if (p.forward_rows != 0 && p.forward_rows != 1) return false;
  if (p.reuse_forward != 0 && p.reuse_forward != 1) return false;
  if (p.reuse_forward == 1 && p.forward_rows != 0) return false;
  if (p.schedule != DRK_SCHEDULE_DYNAMIC && p.schedule != DRK_SCHEDULE_STATIC) return false;
  if (p.n_dw_chunk_events < 0 || (p.dw_chunk_events == nullptr && p.n_dw_chunk_events != 0)) return false;
  if (std::isnan(p.mrs_lo) || std::isnan(p.mrs_hi) || std::isnan(p.veto_ratio)) return false;
  if (p.norm == DRK_NORM_EXPLICIT && !std::isfinite(p.explicit_scale)) return false;
  return true;
}

UmmaFwdArgs umma_fwd_args(const void* hidden, const void* W, const int32_t* ids, int64_t T, int H, int V, int engine,
                          const FwdWs& w, float* logp, float* lse, float* entropy, uint32_t* status,
                          const __nv_bfloat16* hidden_c, const int32_t* rowmap, const int32_t* n_rows, int id_off,
                          float* stats, bool dynamic = true) {
  UmmaFwdArgs a{hidden, W, ids, T, H, V, logp, lse, w.part, w.tgt, w.nsplit, status, umma_ctas(engine), entropy,
                hidden_c, rowmap, n_rows};
  a.id_off = id_off; a.stats = stats;
  a.sched = dynamic ? w.sched : nullptr;
  return a;
}

int run_fwd(const void* hidden, const void* W, int in_dtype, const int32_t* ids, int64_t T, int H, int V,
            bool simt, int engine, const FwdWs& w, float* logp, float* lse, float* entropy, uint32_t* status,
            cudaStream_t st, const __nv_bfloat16* hidden_c = nullptr, const int32_t* rowmap = nullptr,
            const int32_t* n_rows = nullptr, int id_off = 0, float* stats = nullptr) {
  if (simt) {
    SimtFwdArgs a{hidden, W, in_dtype, ids, T, H, V, logp, lse, w.part, w.tgt, w.nsplit, status, entropy};
    a.id_off = id_off; a.stats = stats;
    return launch_simt_fwd(a, st);
  }
  // plan (host only: kernel attributes, tensor maps) first, then enqueue
  UmmaFwdPlan plan;
  int rc = plan_umma_fwd(umma_fwd_args(hidden, W, ids, T, H, V, engine, w, logp, lse, entropy, status, hidden_c, rowmap,
                                       n_rows, id_off, stats), &plan);
  if (rc != DRK_OK) return rc;
  return enqueue_umma_fwd(plan, st);
}

// Vocabulary-range mode of the fused call: log-probs come from all ranges' statistics instead of a forward
// pass, and W holds columns [v_begin, v_begin + V) of a vocabulary of V_total columns.
struct ShardCtx {
  const float* stats_all; int n_shards; int v_begin; int V_total;
};

bool shard_ok(int V_local, int v_begin, int V_total) {
  return V_local >= 1 && v_begin >= 0 && V_total >= 1 && V_total <= (1 << 24) &&
         (int64_t)v_begin + V_local <= V_total;
}

int loss_fwd_bwd_impl(const void* hidden, const void* W, int32_t in_dtype, const int32_t* ids,
                      const float* rollout_logp, const uint8_t* loss_mask, const int32_t* cu_seqlens,
                      const float* seg_adv, int64_t T, int32_t H, int32_t V, int32_t S, const drk_pg_params* pp,
                      float* loss, float* logp, float* lse, float* entropy, float* seg_w, uint8_t* seg_keep,
                      int64_t* counters, void* dH, void* dW, void* workspace, size_t workspace_bytes, uint32_t* status,
                      void* stream, const ShardCtx* sh) {
  g_launches = 0;
  drk_pg_params p;
  if (pp) p = *pp; else drk_pg_params_default(&p);
  if (!sizes_ok(T, H, V, in_dtype) || S < 0 || S > (1 << 24) || !params_ok(p)) return DRK_ERR_INVALID_ARG;
  if (!W || !dW || !loss || !counters || !workspace || !status) return DRK_ERR_INVALID_ARG;
  if (T > 0 && (!hidden || !ids || !rollout_logp || !loss_mask || !logp || !lse || !dH)) return DRK_ERR_INVALID_ARG;
  if (S > 0 && (!cu_seqlens || !seg_adv || !seg_w || !seg_keep)) return DRK_ERR_INVALID_ARG;
  if (!aligned(hidden, 16) || !aligned(W, 16) || !aligned(dH, 16) || !aligned(dW, 16) || !aligned(workspace, 256) ||
      !aligned(logp, 16) || !aligned(rollout_logp, 16) || !aligned(loss_mask, 4))
    return DRK_ERR_INVALID_ARG;
  if (sh != nullptr) {
    if (!shard_ok(V, sh->v_begin, sh->V_total) || sh->n_shards < 1 || sh->n_shards > 4096) return DRK_ERR_INVALID_ARG;
    if (T > 0 && (!sh->stats_all || !aligned(sh->stats_all, 16))) return DRK_ERR_INVALID_ARG;
    if (p.forward_rows != 0) return DRK_ERR_UNSUPPORTED;   // there is no forward pass to restrict
  }
  const bool simt = use_simt(in_dtype, p.engine);
  if (!simt && (H % 8) != 0) return DRK_ERR_UNSUPPORTED;
  if (workspace_bytes < drk_pg_workspace_bytes(T, H, V, S, in_dtype, &p, 1)) return DRK_ERR_WORKSPACE;
  if (p.dw_chunk_events != nullptr) {
    const int vc = round_vchunk(p.v_chunk, T, H, V, simt);
    if (T == 0 || p.n_dw_chunk_events != (int)ceil_div(V, vc)) return DRK_ERR_INVALID_ARG;
    for (int i = 0; i < p.n_dw_chunk_events; ++i)
      if (p.dw_chunk_events[i] == nullptr) return DRK_ERR_INVALID_ARG;
  }
  int rc = check_arch();
  if (rc != DRK_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  Carver c(workspace);
  const FwdWs fw = carve_fwd(c, T, V, simt, p.engine);
  const BwdWs bw = carve_bwd(c, T, H, V, S, simt, p);
  const int id_off = sh ? sh->v_begin : 0;

  auto fail = [&](int code) { g_launches = 0; return code; };

  // Tensor-core path: every host step that can fail (driver entry point, kernel attributes, all tensor maps
  // of the forward and of every vocabulary chunk of the backward) runs here, before the first enqueue.
  const bool fwd_here = T > 0 && sh == nullptr && p.reuse_forward == 0;
  const bool fwd_rows = fwd_here && p.forward_rows == 1 && !simt;
  UmmaFwdPlan fplan;
  UmmaBwdPlan bplan;
  if (!simt && T > 0) {
    if (fwd_here) {
      rc = plan_umma_fwd(umma_fwd_args(hidden, W, ids, T, H, V, p.engine, fw, logp, lse, entropy, status,
                                       fwd_rows ? bw.hidden_c : nullptr, fwd_rows ? bw.rowmap : nullptr,
                                       fwd_rows ? bw.n_rows : nullptr, 0, nullptr,
                                       p.schedule == DRK_SCHEDULE_DYNAMIC), &fplan);
      if (rc != DRK_OK) return fail(rc);
    }
    UmmaBwdArgs b{hidden, W, ids, T, H, V, lse, bw.coeff, static_cast<__nv_bfloat16*>(bw.dL), bw.vc,
                  dH, p.dh_dtype, bw.dH_acc, dW, p.dw_dtype, p.dw_accumulate, status, umma_ctas(p.engine),
                  bw.hidden_c, bw.rowmap, bw.n_rows, p.dw_chunk_events};
    b.id_off = id_off;
    b.sched = p.schedule == DRK_SCHEDULE_DYNAMIC ? bw.sched : nullptr;
    rc = plan_umma_bwd(b, &bplan);
    if (rc != DRK_OK) return fail(rc);
  }

  Range call_range(sh ? "drk_pg_shard_loss_bwd" : "drk_pg_loss_fwd_bwd");
  if (T > 0 && sh == nullptr && p.reuse_forward == 1) {
    // logp and lse come from an earlier forward over the same operands
  } else if (T > 0 && sh != nullptr) {
    Range r("drk: recombine range statistics");
    rc = launch_shard_merge(sh->stats_all, sh->n_shards, ids, T, sh->V_total, logp, lse, entropy, status, st);
    if (rc != DRK_OK) return fail(rc);
  } else if (T > 0 && p.forward_rows == 1 && !simt) {
    // forward over the rows the loss can use: loss-masked tokens inside segments; the rest read 0
    Range r("drk: forward (usable rows)");
    rc = launch_need_rows(loss_mask, cu_seqlens, T, S, bw.coeff, st);
    if (rc != DRK_OK) return fail(rc);
    CompactArgs ca{bw.coeff, static_cast<const __nv_bfloat16*>(hidden), T, H, bw.blk_cnt, bw.blk_off, bw.n_rows,
                   bw.rowmap, bw.hidden_c, status};
    rc = launch_compact(ca, st);
    if (rc != DRK_OK) return fail(rc);
    if (cudaMemsetAsync(logp, 0, sizeof(float) * (size_t)T, st) != cudaSuccess ||
        cudaMemsetAsync(lse, 0, sizeof(float) * (size_t)T, st) != cudaSuccess ||
        (entropy && cudaMemsetAsync(entropy, 0, sizeof(float) * (size_t)T, st) != cudaSuccess))
      return fail(DRK_ERR_CUDA);
    rc = enqueue_umma_fwd(fplan, st);
    if (rc != DRK_OK) return fail(rc);
  } else if (T > 0) {
    Range r("drk: forward");
    rc = simt ? run_fwd(hidden, W, in_dtype, ids, T, H, V, simt, p.engine, fw, logp, lse, entropy, status, st)
              : enqueue_umma_fwd(fplan, st);
    if (rc != DRK_OK) return fail(rc);
  }
  {
    Range r("drk: rejection sampling, coefficients, loss");
    MrsArgs m{};
    m.logp = logp; m.rollout_logp = rollout_logp; m.loss_mask = loss_mask; m.cu = cu_seqlens; m.seg_adv = seg_adv;
    m.T = T; m.S = S;
    m.ln_lo = p.mrs_lo > 0.f ? std::log((double)p.mrs_lo) : -std::numeric_limits<double>::infinity();
    m.ln_hi = std::isinf(p.mrs_hi) ? std::numeric_limits<double>::infinity() : std::log((double)p.mrs_hi);
    m.ln_veto = p.veto_ratio > 0.f ? std::log((double)p.veto_ratio) : -std::numeric_limits<double>::infinity();
    m.norm = p.norm; m.explicit_scale = p.explicit_scale; m.keep_from_caller = p.keep_from_caller;
    m.seg_w = seg_w; m.seg_keep = seg_keep; m.loss = loss; m.counters = counters; m.coeff = bw.coeff;
    m.seg_stats = bw.seg_stats; m.status = status;
    rc = launch_mrs(m, st);
  }
  if (rc != DRK_OK) return fail(rc);
  Range bwd_range("drk: backward");

  if (T == 0) {
    // no tokens: gradients are zero
    if (!p.dw_accumulate) {
      const size_t esz = p.dw_dtype == DRK_BF16 ? 2 : 4;
      if (cudaMemsetAsync(dW, 0, esz * (size_t)V * (size_t)H, st) != cudaSuccess) return fail(DRK_ERR_CUDA);
    }
    return DRK_OK;
  }
  if (simt) {
    SimtBwdArgs b{hidden, W, in_dtype, ids, T, H, V, lse, bw.coeff, static_cast<float*>(bw.dL), bw.vc,
                  dH, p.dh_dtype, bw.dH_acc, dW, p.dw_dtype, p.dw_accumulate, p.dw_chunk_events};
    b.id_off = id_off;
    rc = launch_simt_bwd(b, st);
  } else {
    CompactArgs ca{bw.coeff, static_cast<const __nv_bfloat16*>(hidden), T, H, bw.blk_cnt, bw.blk_off, bw.n_rows,
                   bw.rowmap, bw.hidden_c, status};
    rc = launch_compact(ca, st);
    if (rc != DRK_OK) return fail(rc);
    rc = enqueue_umma_bwd(bplan, st);
  }
  if (rc != DRK_OK) return fail(rc);
  return DRK_OK;
}

}  // namespace
}  // namespace drk

using namespace drk;

extern "C" {

void drk_pg_params_default(drk_pg_params* p) {
  if (!p) return;
  p->mrs_lo = 0.999f;
  p->mrs_hi = 1.001f;
  p->veto_ratio = 1e-4f;
  p->norm = DRK_NORM_KEPT_TOKENS;
  p->explicit_scale = 1.0f;
  p->dw_dtype = DRK_F32;
  p->dh_dtype = DRK_F32;
  p->dw_accumulate = 0;
  p->engine = DRK_ENGINE_AUTO;
  p->v_chunk = 0;
  p->keep_from_caller = 0;
  p->forward_rows = 0;
  p->dw_chunk_events = nullptr;
  p->n_dw_chunk_events = 0;
  p->reuse_forward = 0;
  p->schedule = DRK_SCHEDULE_DYNAMIC;
}

int drk_pg_bwd_chunks(int64_t T, int32_t H, int32_t V, int32_t in_dtype, const drk_pg_params* pp, int32_t* v_chunk) {
  drk_pg_params p;
  if (pp) p = *pp; else drk_pg_params_default(&p);
  if (!sizes_ok(T, H, V, in_dtype) || !params_ok(p) || !v_chunk) return DRK_ERR_INVALID_ARG;
  const int vc = round_vchunk(p.v_chunk, T, H, V, use_simt(in_dtype, p.engine));
  *v_chunk = vc;
  return (int)ceil_div(V, vc);
}

size_t drk_pg_workspace_bytes(int64_t T, int32_t H, int32_t V, int32_t S, int32_t in_dtype,
                              const drk_pg_params* pp, int32_t which) {
  drk_pg_params p;
  if (pp) p = *pp; else drk_pg_params_default(&p);
  if (!sizes_ok(T, H, V, in_dtype) || S < 0 || !params_ok(p) || (which != 0 && which != 1)) return 0;
  const bool simt = use_simt(in_dtype, p.engine);
  Carver c(nullptr);
  carve_fwd(c, T, V, simt, p.engine);
  if (which == 1) carve_bwd(c, T, H, V, S, simt, p);
  return c.off + 256;  // never 0 for valid arguments
}

int drk_trloo_advantage(const float* reward, const uint8_t* valid, const int32_t* prompt_of_rollout, int32_t R,
                        int32_t Tmax, float gamma, int32_t baseline, float* ret, float* adv, int32_t* gsize,
                        uint32_t* status, void* stream) {
  g_launches = 0;
  if (R < 0 || Tmax < 0) return DRK_ERR_INVALID_ARG;
  if (baseline != DRK_BASELINE_TRLOO && baseline != DRK_BASELINE_GRPO) return DRK_ERR_INVALID_ARG;
  if (!(gamma >= 0.f && gamma <= 1.f)) return DRK_ERR_INVALID_ARG;
  if (Tmax > 64) return DRK_ERR_UNSUPPORTED;
  if (R == 0 || Tmax == 0) return DRK_OK;
  if (!reward || !valid || !prompt_of_rollout || !ret || !adv || !gsize) return DRK_ERR_INVALID_ARG;
  int rc = check_arch();
  if (rc != DRK_OK) return rc;
  rc = launch_trloo(reward, valid, prompt_of_rollout, R, Tmax, gamma, baseline, ret, adv, gsize, status,
                    static_cast<cudaStream_t>(stream));
  if (rc != DRK_OK) g_launches = 0;
  return rc;
}

int drk_pg_logprob_fwd(const void* hidden, const void* W, int32_t in_dtype, const int32_t* ids, int64_t T,
                       int32_t H, int32_t V, int32_t engine, float* logp, float* lse, float* entropy, void* workspace,
                       size_t workspace_bytes, uint32_t* status, void* stream) {
  g_launches = 0;
  if (!sizes_ok(T, H, V, in_dtype)) return DRK_ERR_INVALID_ARG;
  if (!engine_ok(engine)) return DRK_ERR_INVALID_ARG;
  if (T == 0) return DRK_OK;
  if (!hidden || !W || !ids || !logp || !lse || !workspace || !status) return DRK_ERR_INVALID_ARG;
  if (!aligned(hidden, 16) || !aligned(W, 16) || !aligned(workspace, 256)) return DRK_ERR_INVALID_ARG;
  const bool simt = use_simt(in_dtype, engine);
  if (!simt && (H % 8) != 0) return DRK_ERR_UNSUPPORTED;
  drk_pg_params p;
  drk_pg_params_default(&p);
  p.engine = engine;
  if (workspace_bytes < drk_pg_workspace_bytes(T, H, V, 0, in_dtype, &p, 0)) return DRK_ERR_WORKSPACE;
  int rc = check_arch();
  if (rc != DRK_OK) return rc;
  Carver c(workspace);
  const FwdWs w = carve_fwd(c, T, V, simt, engine);
  rc = run_fwd(hidden, W, in_dtype, ids, T, H, V, simt, engine, w, logp, lse, entropy, status,
               static_cast<cudaStream_t>(stream));
  if (rc != DRK_OK) g_launches = 0;
  return rc;
}

int drk_pg_loss_fwd_bwd(const void* hidden, const void* W, int32_t in_dtype, const int32_t* ids,
                        const float* rollout_logp, const uint8_t* loss_mask, const int32_t* cu_seqlens,
                        const float* seg_adv, int64_t T, int32_t H, int32_t V, int32_t S, const drk_pg_params* pp,
                        float* loss, float* logp, float* lse, float* entropy, float* seg_w, uint8_t* seg_keep,
                        int64_t* counters, void* dH, void* dW, void* workspace, size_t workspace_bytes, uint32_t* status,
                        void* stream) {
  return loss_fwd_bwd_impl(hidden, W, in_dtype, ids, rollout_logp, loss_mask, cu_seqlens, seg_adv, T, H, V, S, pp, loss,
                           logp, lse, entropy, seg_w, seg_keep, counters, dH, dW, workspace, workspace_bytes, status,
                           stream, nullptr);
}

int drk_pg_shard_stats_fwd(const void* hidden, const void* W_shard, int32_t in_dtype, const int32_t* ids, int64_t T,
                           int32_t H, int32_t V_local, int32_t v_begin, int32_t V_total, int32_t engine, float* stats,
                           void* workspace, size_t workspace_bytes, uint32_t* status, void* stream) {
  g_launches = 0;
  if (!sizes_ok(T, H, V_local, in_dtype) || !shard_ok(V_local, v_begin, V_total)) return DRK_ERR_INVALID_ARG;
  if (!engine_ok(engine)) return DRK_ERR_INVALID_ARG;
  if (T == 0) return DRK_OK;
  if (!hidden || !W_shard || !ids || !stats || !workspace || !status) return DRK_ERR_INVALID_ARG;
  if (!aligned(hidden, 16) || !aligned(W_shard, 16) || !aligned(stats, 16) || !aligned(workspace, 256))
    return DRK_ERR_INVALID_ARG;
  const bool simt = use_simt(in_dtype, engine);
  if (!simt && (H % 8) != 0) return DRK_ERR_UNSUPPORTED;
  drk_pg_params p;
  drk_pg_params_default(&p);
  p.engine = engine;
  if (workspace_bytes < drk_pg_workspace_bytes(T, H, V_local, 0, in_dtype, &p, 0)) return DRK_ERR_WORKSPACE;
  int rc = check_arch();
  if (rc != DRK_OK) return rc;
  Carver c(workspace);
  const FwdWs w = carve_fwd(c, T, V_local, simt, engine);
  rc = run_fwd(hidden, W_shard, in_dtype, ids, T, H, V_local, simt, engine, w, nullptr, nullptr, nullptr, status,
               static_cast<cudaStream_t>(stream), nullptr, nullptr, nullptr, v_begin, stats);
  if (rc != DRK_OK) g_launches = 0;
  return rc;
}

int drk_pg_shard_merge(const float* stats_all, int32_t n_shards, const int32_t* ids, int64_t T, int32_t V_total,
                       float* logp, float* lse, float* entropy, uint32_t* status, void* stream) {
  g_launches = 0;
  if (T < 0 || T > (1 << 24) || V_total < 1 || V_total > (1 << 24) || n_shards < 1 || n_shards > 4096)
    return DRK_ERR_INVALID_ARG;
  if (T == 0) return DRK_OK;
  if (!stats_all || !ids || !logp || !lse || !status || !aligned(stats_all, 16)) return DRK_ERR_INVALID_ARG;
  int rc = check_arch();
  if (rc != DRK_OK) return rc;
  rc = launch_shard_merge(stats_all, n_shards, ids, T, V_total, logp, lse, entropy, status,
                          static_cast<cudaStream_t>(stream));
  if (rc != DRK_OK) g_launches = 0;
  return rc;
}

int drk_pg_shard_loss_bwd(const void* hidden, const void* W_shard, int32_t in_dtype, const int32_t* ids,
                          const float* stats_all, int32_t n_shards, const float* rollout_logp,
                          const uint8_t* loss_mask, const int32_t* cu_seqlens, const float* seg_adv, int64_t T,
                          int32_t H, int32_t V_local, int32_t v_begin, int32_t V_total, int32_t S,
                          const drk_pg_params* p, float* loss, float* logp, float* lse, float* entropy, float* seg_w,
                          uint8_t* seg_keep, int64_t* counters, void* dH_part, void* dW_shard, void* workspace,
                          size_t workspace_bytes, uint32_t* status, void* stream) {
  const ShardCtx sh{stats_all, n_shards, v_begin, V_total};
  return loss_fwd_bwd_impl(hidden, W_shard, in_dtype, ids, rollout_logp, loss_mask, cu_seqlens, seg_adv, T, H, V_local,
                           S, p, loss, logp, lse, entropy, seg_w, seg_keep, counters, dH_part, dW_shard, workspace,
                           workspace_bytes, status, stream, &sh);
}

int drk_segment_advantages(const float* adv, const int32_t* seg_rollout, const int32_t* seg_turn, int32_t R,
                           int32_t Tmax, int32_t S, float* seg_adv, uint32_t* status, void* stream) {
  g_launches = 0;
  if (R < 0 || Tmax < 0 || S < 0) return DRK_ERR_INVALID_ARG;
  if (S == 0) return DRK_OK;
  if (!seg_rollout || !seg_turn || !seg_adv || !status || (!adv && (int64_t)R * Tmax > 0)) return DRK_ERR_INVALID_ARG;
  int rc = check_arch();
  if (rc != DRK_OK) return rc;
  rc = launch_segment_advantages(adv, seg_rollout, seg_turn, R, Tmax, S, seg_adv, status,
                                 static_cast<cudaStream_t>(stream));
  if (rc != DRK_OK) g_launches = 0;
  return rc;
}

int drk_selftest_bounded_wait(uint32_t limit_ms, uint32_t* status, uint64_t* waited_ns, void* stream) {
  g_launches = 0;
  if (limit_ms < 1 || limit_ms > 1000 || !status || !waited_ns) return DRK_ERR_INVALID_ARG;
  int rc = check_arch();
  if (rc != DRK_OK) return rc;
  rc = launch_bounded_wait_selftest(limit_ms, status, waited_ns, static_cast<cudaStream_t>(stream));
  if (rc != DRK_OK) g_launches = 0;
  return rc;
}

int drk_last_launch_count(void) { return g_launches; }

uint64_t drk_tensor_map_encodes(void) { return umma_map_encodes(); }

void drk_selftest_fail_tensor_map(int32_t nth) { umma_fail_map_request(nth); }

const char* drk_status_string(int s) {
  switch (s) {
    case DRK_OK: return "ok";
    case DRK_ERR_INVALID_ARG: return "invalid argument";
    case DRK_ERR_UNSUPPORTED: return "unsupported shape";
    case DRK_ERR_WORKSPACE: return "workspace too small";
    case DRK_ERR_CUDA: return "CUDA call failed";
    case DRK_ERR_ARCH: return "device is not sm_100";
    default: return "unknown status";
  }
}

int drk_version(void) { return 101; }

int drk_bounds_checked(void) {
#ifdef DRK_BOUNDS_CHECK
  return 1;
#else
  return 0;
#endif
}

}  // extern "C"
