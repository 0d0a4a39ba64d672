// Shared host/device helpers of the drk library (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/drk.h"

namespace drk {

// Per-thread count of kernels enqueued by the running entry point.
extern thread_local int g_launches;

#define DRK_CUDA_CHECK(expr)                      \
  do {                                            \
    cudaError_t e__ = (expr);                     \
    if (e__ != cudaSuccess) return DRK_ERR_CUDA;  \
  } while (0)

// Call after every kernel launch: counts it and maps launch errors.
#define DRK_LAUNCHED()                                  \
  do {                                                  \
    ++::drk::g_launches;                                \
    if (cudaGetLastError() != cudaSuccess) return DRK_ERR_CUDA; \
  } while (0)

// Multiprocessors of the current device (148 on B200; the same number when no device can be queried, so that
// size queries still answer on a host without a GPU).  Grids, wave models and split counts derive from it.
int sm_count();

// Checked build (-DDRK_BOUNDS_CHECK): every index that a kernel derives from device-side data (row maps,
// compacted counts, work-unit numbers, token ids used as addresses) is range-checked before use; a violation
// sets DRK_STATUS_BOUNDS in the status word and the access is skipped -- no trap, no fault.  In the ordinary
// build the test folds to `true` and costs nothing.
#ifdef DRK_BOUNDS_CHECK
#define DRK_IN_RANGE(cond, status_ptr) ((cond) ? true : (atomicOr((status_ptr), DRK_STATUS_BOUNDS), false))
#else
#define DRK_IN_RANGE(cond, status_ptr) (true)
#endif

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

// Token id relative to the vocabulary range [id_off, id_off + width): the local column, or -1 when the
// token belongs to another range (or is invalid).
__device__ __forceinline__ int local_id(int id, int id_off, int width) {
  const uint32_t rel = (uint32_t)id - (uint32_t)id_off;
  return rel < (uint32_t)width ? (int)rel : -1;
}

// ---- internal launchers (each returns a drk_status) -------------------------------------------

int launch_trloo(const float* reward, const uint8_t* valid, const int32_t* prompt, int R, int Tmax,
                 float gamma, int baseline, float* ret, float* adv, int32_t* gsize, uint32_t* status,
                 cudaStream_t st);

// Per-segment statistics, rejection decision, coefficients and loss.
struct MrsArgs {
  const float* logp; const float* rollout_logp; const uint8_t* loss_mask; const int32_t* cu;
  const float* seg_adv; int64_t T; int S;
  double ln_lo, ln_hi, ln_veto; int norm; float explicit_scale; int keep_from_caller;
  float* seg_w; uint8_t* seg_keep; float* loss; int64_t* counters; float* coeff /*[T]*/;
  double* seg_stats /*[S*4] workspace*/; uint32_t* status;
};
int launch_mrs(const MrsArgs& a, cudaStream_t st);
// seg_adv[g] = adv[seg_rollout[g] * Tmax + seg_turn[g]] (0 and a status bit for indices outside the table)
int launch_segment_advantages(const float* adv, const int32_t* seg_rollout, const int32_t* seg_turn, int R, int Tmax,
                              int S, float* seg_adv, uint32_t* status, cudaStream_t st);

// FFMA path.
struct SimtFwdArgs {
  const void* hidden; const void* W; int in_dtype; const int32_t* ids; int64_t T; int H; int V;
  float* logp; float* lse; float* part /*[nsplit*T*4]*/; float* tgt /*[T]*/; int nsplit; uint32_t* status;
  float* entropy /*[T] or null*/;
  // vocabulary-range mode: W holds columns [id_off, id_off + V) of a larger vocabulary; when stats is
  // given the call ends with the range's per-row statistics [T,4] instead of logp / lse
  int id_off = 0; float* stats = nullptr;
};
int simt_nsplit(int64_t T, int V);
int launch_simt_fwd(const SimtFwdArgs& a, cudaStream_t st);
int launch_lse_merge(const float* part, const float* tgt, const int32_t* ids, int64_t T, int V, int nsplit,
                     float* logp, float* lse, float* entropy, uint32_t* status, const int32_t* rowmap,
                     const int32_t* n_rows, cudaStream_t st);
// Vocabulary-range mode: per-row statistics (max, sum-exp, sum-exp-times-logit, target logit or 0) of one
// range from its partials, and the recombination of all ranges' statistics into logp, lse, entropy.
int launch_shard_stats(const float* part, const float* tgt, const int32_t* ids, int id_off, int64_t T, int V,
                       int nsplit, float* stats, uint32_t* status, cudaStream_t st);
int launch_shard_merge(const float* stats_all, int n_shards, const int32_t* ids, int64_t T, int V_total, float* logp,
                       float* lse, float* entropy, uint32_t* status, cudaStream_t st);
struct SimtBwdArgs {
  const void* hidden; const void* W; int in_dtype; const int32_t* ids; int64_t T; int H; int V;
  const float* lse; const float* coeff; float* dL /*[T*vc] fp32 workspace*/; int vc;
  void* dH; int dh_dtype; float* dH_acc /*fp32 [T,H] or null when dH is fp32*/;
  void* dW; int dw_dtype; int dw_accumulate;
  void* const* chunk_events;  // optional cudaEvent_t per vocabulary chunk, recorded when its dW rows are final
  int id_off = 0;             // W holds columns [id_off, id_off + V) of a larger vocabulary
};
int launch_simt_bwd(const SimtBwdArgs& a, cudaStream_t st);

// tcgen05 path (bf16 inputs).
struct UmmaFwdArgs {
  const void* hidden; const void* W; const int32_t* ids; int64_t T; int H; int V;
  float* logp; float* lse; float* part /*[nsplit*T*4]*/; float* tgt; int nsplit; uint32_t* status;
  int ctas /*1: one CTA per tile; 2: CTA pairs*/;
  float* entropy /*[T] or null*/;
  // optional: evaluate only the rows listed in rowmap (gathered into hidden_c); others are left untouched
  const __nv_bfloat16* hidden_c; const int32_t* rowmap; const int32_t* n_rows;
  int id_off = 0; float* stats = nullptr;   // vocabulary-range mode, as in SimtFwdArgs
  int32_t* sched = nullptr;                 // one work counter (dynamic schedule) or null (static)
};
int umma_nsplit(int64_t T, int V, int ctas, bool frugal);
int launch_umma_fwd(const UmmaFwdArgs& a, cudaStream_t st);
struct UmmaBwdArgs {
  const void* hidden; const void* W; const int32_t* ids; int64_t T; int H; int V;
  const float* lse; const float* coeff; __nv_bfloat16* dL /*[T*vc]*/; int vc;
  void* dH; int dh_dtype; float* dH_acc /*fp32 [ceil256(T), H]: accumulator over the compacted rows*/;
  void* dW; int dw_dtype; int dw_accumulate; uint32_t* status;
  int ctas;
  const __nv_bfloat16* hidden_c; const int32_t* rowmap; const int32_t* n_rows;  // compacted rows
  void* const* chunk_events;  // optional cudaEvent_t per vocabulary chunk, recorded when its dW rows are final
  int id_off = 0;             // W holds columns [id_off, id_off + V) of a larger vocabulary
  int32_t* sched = nullptr;   // three work counters per vocabulary chunk (dynamic schedule) or null (static)
};
int launch_umma_bwd(const UmmaBwdArgs& a, cudaStream_t st);

// Compaction of the rows with non-zero coefficient (backward pass of the tensor-core path).
struct CompactArgs {
  const float* coeff; const __nv_bfloat16* hidden; int64_t T; int H;
  int32_t* blk_cnt; int32_t* blk_off; int32_t* n_rows /*[2]: count, count rounded up to 256*/;
  int32_t* rowmap /*[compact_map_len(T)]*/; __nv_bfloat16* hidden_c /*[compact_map_len(T), H]*/;
  uint32_t* status = nullptr;   // status word for the checked build's range checks
};
int64_t compact_map_len(int64_t T);
int compact_blocks(int64_t T);
int launch_compact(const CompactArgs& a, cudaStream_t st);
// dst[rowmap[r], :] = src[r, :] for the n_rows[0] compacted rows; src fp32 [*, H], dst fp32 or bf16 [T, H]
int launch_scatter_rows(const float* src, int H, const int32_t* rowmap, const int32_t* n_rows, void* dst, bool dst_bf16,
                        int64_t T, uint32_t* status, cudaStream_t st);
// need[t] = 1 for loss-masked tokens inside a segment, else 0 (the rows whose log-prob the loss can use)
int launch_need_rows(const uint8_t* loss_mask, const int32_t* cu, int64_t T, int S, float* need, cudaStream_t st);

int launch_bounded_wait_selftest(uint32_t limit_ms, uint32_t* status, uint64_t* waited_ns, cudaStream_t st);

// Small utility kernels.
int launch_f32_to_bf16(const float* src, __nv_bfloat16* dst, size_t n, cudaStream_t st);

}  // namespace drk
