// drk_pg_logprob_fwd_noalloc: the forward log-prob call for callers that cannot provide a workspace.
//
// The ordinary call keeps its per-row partial (max, sum-exp) pairs and target logits in a workspace
// that the caller allocates.  Some callers have no way to allocate at call time: a training loop whose
// framework has already handed all device memory to its own pool, or a latency-critical section
// where cudaMalloc's implicit device-wide synchronisation is not acceptable.  For them the same
// kernels run here with that scratch placed in a fixed array that is part of the library image.
//
// Consequences of the fixed array, all of which the header documents too:
//   - every GPU that loads the library holds DRK_NOALLOC_SCRATCH_BYTES until the process exits;
//   - sizes that need more are rejected with DRK_ERR_WORKSPACE, nothing is enqueued;
//   - all calls on a device share the array, so two calls whose kernels may overlap on the GPU
//     (different streams without ordering) race; calls on one stream are safe;
//   - the array keeps the previous call's contents.  Every partial that the merge step reads is
//     rewritten by the call itself; the target-logit slots are cleared first, so a row whose id is
//     invalid can never pick up a stale value;
//   - the first call on each device looks up the array's device address (cudaGetSymbolAddress),
//     which may initialise the context for that symbol: make that first call outside any stream
//     capture.
// No cudaMalloc, cudaFree or allocating library routine is called.
#include "common.cuh"
#include "umma_plan.cuh"
#include <mutex>

namespace drk {
namespace {

constexpr size_t kScratchBytes = DRK_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Device storage.  In host code this name is only a handle for the runtime's symbol table, never a
// device address: the address is fetched once per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the array on the current device; looked up on first use.
int scratch_address(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return DRK_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return DRK_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return DRK_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return DRK_OK;
}

}  // namespace
}  // namespace drk

using namespace drk;

extern "C" int drk_pg_logprob_fwd_noalloc(const void* hidden, const void* W, int32_t in_dtype, const int32_t* ids,
                                          int64_t T, int32_t H, int32_t V, int32_t engine, float* logp, float* lse,
                                          uint32_t* status, void* stream) {
  g_launches = 0;
  if (T < 0 || T > (1 << 24) || H < 1 || H > 65536 || V < 1 || V > (1 << 24)) return DRK_ERR_INVALID_ARG;
  if (in_dtype != DRK_F32 && in_dtype != DRK_BF16) return DRK_ERR_INVALID_ARG;
  if (engine != DRK_ENGINE_AUTO && engine != DRK_ENGINE_SIMT && engine != DRK_ENGINE_UMMA_1CTA) return DRK_ERR_INVALID_ARG;
  if (T == 0) return DRK_OK;
  if (!hidden || !W || !ids || !logp || !lse || !status) return DRK_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(hidden) % 16 || reinterpret_cast<uintptr_t>(W) % 16) return DRK_ERR_INVALID_ARG;
  const bool simt = (in_dtype == DRK_F32) || (engine == DRK_ENGINE_SIMT);
  if (!simt && (H % 8) != 0) return DRK_ERR_UNSUPPORTED;

  // scratch layout: partials [nsplit, T, 4] floats, target logits [T] floats, one work counter; each 256-aligned
  const int ctas = engine == DRK_ENGINE_UMMA_1CTA ? 1 : 2;
  const int nsplit = simt ? simt_nsplit(T, V) : umma_nsplit(T, V, ctas, true);
  const size_t part_bytes = align_up(sizeof(float) * 4 * (size_t)nsplit * (size_t)T, 256);
  const size_t tgt_bytes = align_up(sizeof(float) * (size_t)T, 256);
  const size_t sched_bytes = 256;   // the forward kernel's work counter (cleared by the launch code)
  if (part_bytes + tgt_bytes + sched_bytes > kScratchBytes) return DRK_ERR_WORKSPACE;

  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return DRK_ERR_CUDA;
  if (major != 10) return DRK_ERR_ARCH;

  void* base = nullptr;
  int rc = scratch_address(&base);
  if (rc != DRK_OK) return rc;
  float* part = reinterpret_cast<float*>(base);
  float* tgt = reinterpret_cast<float*>(static_cast<char*>(base) + part_bytes);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  UmmaFwdPlan plan;
  if (!simt) {   // kernel attributes and tensor maps (host only) before anything is enqueued
    UmmaFwdArgs a{hidden, W, ids, T, H, V, logp, lse, part, tgt, nsplit, status, ctas, nullptr, nullptr, nullptr, nullptr};
    a.sched = reinterpret_cast<int32_t*>(static_cast<char*>(base) + part_bytes + tgt_bytes);
    rc = plan_umma_fwd(a, &plan);
    if (rc != DRK_OK) return rc;
  }
  if (cudaMemsetAsync(tgt, 0, tgt_bytes, st) != cudaSuccess) return DRK_ERR_CUDA;

  if (simt) {
    SimtFwdArgs a{hidden, W, in_dtype, ids, T, H, V, logp, lse, part, tgt, nsplit, status, nullptr};
    rc = launch_simt_fwd(a, st);
  } else {
    rc = enqueue_umma_fwd(plan, st);
  }
  if (rc != DRK_OK) g_launches = 0;
  return rc;
}
