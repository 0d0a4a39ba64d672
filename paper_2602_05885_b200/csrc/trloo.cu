// Reward-to-go returns (Sec. 4.2, Eq. 2) and turn-level advantages (Eq. 5 TRLOO, Eq. 3 GRPO).
//
// One warp per prompt.  Rollouts of a prompt are contiguous, so the warp whose index is the first
// rollout of a run owns that run; every other warp exits at once.  For each turn the warp's lanes
// stride over the run's rollouts, form each return in fp64, and reduce (sum, count) over the valid
// ones with shuffles: a segmented reduction whose segment is the (prompt, turn) group.  The table is
// a few thousand scalars at most, so the kernel is latency-bound and one pass is all there is.
#include "common.cuh"

namespace drk {

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ int warp_sum(int x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// G[i,t] = sum_{t' >= t, valid} gamma^(t'-t) R[i,t'], 0 if (i,t) itself is invalid.
__device__ __forceinline__ double return_at(const float* __restrict__ reward,
                                            const uint8_t* __restrict__ valid, int i, int t, int Tmax,
                                            double gamma) {
  const size_t row = (size_t)i * Tmax;
  if (!valid[row + t]) return 0.0;
  double acc = 0.0, pw = 1.0;
  for (int tp = t; tp < Tmax; ++tp) {
    if (valid[row + tp]) acc += pw * (double)reward[row + tp];
    pw *= gamma;
  }
  return acc;
}

__global__ void trloo_kernel(const float* __restrict__ reward, const uint8_t* __restrict__ valid,
                             const int32_t* __restrict__ prompt, int R, int Tmax, double gamma,
                             int baseline, float* __restrict__ ret, float* __restrict__ adv,
                             int32_t* __restrict__ gsize, uint32_t* __restrict__ status) {
  const int warp = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5);
  const int lane = threadIdx.x & 31;
  if (warp >= R) return;
  const int first = warp;
  const int pid = prompt[first];
  // groups are runs of equal prompt ids; a decrease means some prompt's rollouts are not contiguous
  if (first > 0 && prompt[first - 1] > pid && status != nullptr && lane == 0) atomicOr(status, DRK_STATUS_BAD_GROUPS);
  if (first > 0 && prompt[first - 1] == pid) return;  // not the head of a run
  // find the end of the run: first index whose prompt differs
  int end = first + 1;
  for (;;) {
    const int j = end + lane;
    const bool same = (j < R) && (prompt[j] == pid);
    const unsigned m = __ballot_sync(0xffffffffu, same);
    if (m == 0xffffffffu) { end += 32; continue; }
    end += __ffs(~m) - 1;
    break;
  }
  for (int t = 0; t < Tmax; ++t) {
    // pass 1: group sum and size
    double s = 0.0;
    int n = 0;
    for (int i = first + lane; i < end; i += 32) {
      if (valid[(size_t)i * Tmax + t]) {
        s += return_at(reward, valid, i, t, Tmax, gamma);
        n += 1;
      }
    }
    s = warp_sum(s);
    n = warp_sum(n);
    // pass 2: advantages.  N*G - S is exact in fp64 for fp32-sized inputs, so an all-equal group
    // gives exactly zero.
    for (int i = first + lane; i < end; i += 32) {
      const size_t o = (size_t)i * Tmax + t;
      if (!valid[o]) { ret[o] = 0.f; adv[o] = 0.f; gsize[o] = 0; continue; }
      const double g = return_at(reward, valid, i, t, Tmax, gamma);
      double a;
      if (baseline == DRK_BASELINE_GRPO) {
        a = ((double)n * g - s) / (double)n;                    // G - mean
      } else {
        a = (n > 1) ? ((double)n * g - s) / (double)(n - 1) : 0.0;  // G - mean of the others
      }
      ret[o] = (float)g;
      adv[o] = (float)a;
      gsize[o] = n;
    }
  }
}

int launch_trloo(const float* reward, const uint8_t* valid, const int32_t* prompt, int R, int Tmax,
                 float gamma, int baseline, float* ret, float* adv, int32_t* gsize, uint32_t* status,
                 cudaStream_t st) {
  if (R == 0 || Tmax == 0) return DRK_OK;
  const int threads = 128;  // 4 warps
  const int blocks = (int)ceil_div((int64_t)R * 32, threads);
  trloo_kernel<<<blocks, threads, 0, st>>>(reward, valid, prompt, R, Tmax, (double)gamma, baseline, ret,
                                           adv, gsize, status);
  DRK_LAUNCHED();
  return DRK_OK;
}

// Every turn of a trajectory is one training sample (Sec. 4.3): segment g of a packed micro-batch holds
// turn seg_turn[g] of rollout seg_rollout[g] and takes that entry of the advantage table.
__global__ void segment_advantages_kernel(const float* __restrict__ adv, const int32_t* __restrict__ seg_rollout,
                                          const int32_t* __restrict__ seg_turn, int R, int Tmax, int S,
                                          float* __restrict__ seg_adv, uint32_t* __restrict__ status) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= S) return;
  const int i = seg_rollout[g], t = seg_turn[g];
  if (i < 0 || i >= R || t < 0 || t >= Tmax) {
    seg_adv[g] = 0.f;
    atomicOr(status, DRK_STATUS_BAD_SEGMENTS);
    return;
  }
  seg_adv[g] = adv[(size_t)i * Tmax + t];
}

int launch_segment_advantages(const float* adv, const int32_t* seg_rollout, const int32_t* seg_turn, int R, int Tmax,
                              int S, float* seg_adv, uint32_t* status, cudaStream_t st) {
  if (S == 0) return DRK_OK;
  segment_advantages_kernel<<<(unsigned)ceil_div(S, 256), 256, 0, st>>>(adv, seg_rollout, seg_turn, R, Tmax, S,
                                                                        seg_adv, status);
  DRK_LAUNCHED();
  return DRK_OK;
}

}  // namespace drk
