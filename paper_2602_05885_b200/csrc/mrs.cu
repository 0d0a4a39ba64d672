// Geometric mismatch rejection sampling with token veto (Sec. 5.1) and the REINFORCE surrogate's
// per-token coefficients and loss (App. A).
//
// Three small kernels over the T per-token floats:
//   seg_stats_kernel : one block per training sample (segment); 128-bit loads of logp / rollout_logp
//                      and 32-bit loads of four mask bytes over the aligned body of the segment,
//                      scalar loads for its ragged ends; block reduction of
//                      {masked count, sum delta, min delta, sum logp} in fp64.
//   finalize_kernel  : one block; per segment the decision (in log space, fp64), then the
//                      normaliser, the loss and the counters, reduced in a fixed order.
//   coeff_kernel     : one block per segment writes c_t = mask_t * keep * A * scale.
#include "common.cuh"
#include <math_constants.h>

namespace drk {

constexpr int kStatThreads = 256;

struct SegAcc {
  double sum_delta, sum_logp;
  double min_delta;
  int cnt;
};

__device__ __forceinline__ void acc_token(SegAcc& a, float lp, float rl, uint8_t m) {
  if (m) {
    const double d = (double)lp - (double)rl;
    a.sum_delta += d;
    a.sum_logp += (double)lp;
    a.min_delta = fmin(a.min_delta, d);
    a.cnt += 1;
  }
}

__global__ void __launch_bounds__(kStatThreads)
seg_stats_kernel(const float* __restrict__ logp, const float* __restrict__ rollout_logp,
                 const uint8_t* __restrict__ mask, const int32_t* __restrict__ cu, int64_t T,
                 double* __restrict__ seg_stats, uint32_t* __restrict__ status) {
  const int g = blockIdx.x;
  int64_t a = cu[g], b = cu[g + 1];
  if (a < 0 || b < a || b > T) {
    if (threadIdx.x == 0) atomicOr(status, DRK_STATUS_BAD_SEGMENTS);
    a = b = 0;
  }
  SegAcc acc{0.0, 0.0, CUDART_INF, 0};
  // ragged head up to a multiple of 4, aligned body, ragged tail
  const int64_t body0 = min(b, (a + 3) & ~(int64_t)3);
  const int64_t body1 = max(body0, b & ~(int64_t)3);
  for (int64_t t = a + threadIdx.x; t < body0; t += kStatThreads) acc_token(acc, logp[t], rollout_logp[t], mask[t]);
  for (int64_t t = body0 + 4 * (int64_t)threadIdx.x; t < body1; t += 4 * kStatThreads) {
    const float4 lp = *reinterpret_cast<const float4*>(logp + t);
    const float4 rl = *reinterpret_cast<const float4*>(rollout_logp + t);
    const uchar4 m = *reinterpret_cast<const uchar4*>(mask + t);
    acc_token(acc, lp.x, rl.x, m.x);
    acc_token(acc, lp.y, rl.y, m.y);
    acc_token(acc, lp.z, rl.z, m.z);
    acc_token(acc, lp.w, rl.w, m.w);
  }
  for (int64_t t = body1 + threadIdx.x; t < b; t += kStatThreads) acc_token(acc, logp[t], rollout_logp[t], mask[t]);

#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    acc.sum_delta += __shfl_xor_sync(0xffffffffu, acc.sum_delta, o);
    acc.sum_logp += __shfl_xor_sync(0xffffffffu, acc.sum_logp, o);
    acc.min_delta = fmin(acc.min_delta, __shfl_xor_sync(0xffffffffu, acc.min_delta, o));
    acc.cnt += __shfl_xor_sync(0xffffffffu, acc.cnt, o);
  }
  __shared__ SegAcc sh[kStatThreads / 32];
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    SegAcc r = sh[0];
    for (int w = 1; w < kStatThreads / 32; ++w) {
      r.sum_delta += sh[w].sum_delta;
      r.sum_logp += sh[w].sum_logp;
      r.min_delta = fmin(r.min_delta, sh[w].min_delta);
      r.cnt += sh[w].cnt;
    }
    double* o = seg_stats + 4 * (size_t)g;
    o[0] = (double)r.cnt;
    o[1] = r.sum_delta;
    o[2] = r.min_delta;
    o[3] = r.sum_logp;
  }
}

constexpr int kFinThreads = 256;

// Fixed-order block reduction of one double and three 64-bit counts.
__device__ double block_sum(double x, double* sh) {
  sh[threadIdx.x] = x;
  __syncthreads();
  for (int s = kFinThreads / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
    __syncthreads();
  }
  const double r = sh[0];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kFinThreads)
finalize_kernel(double* __restrict__ seg_stats, const float* __restrict__ seg_adv, int S, double ln_lo,
                double ln_hi, double ln_veto, int norm, float explicit_scale, int keep_from_caller,
                float* __restrict__ seg_w,
                uint8_t* __restrict__ seg_keep, float* __restrict__ loss, int64_t* __restrict__ counters) {
  __shared__ double sh[kFinThreads];
  double kept_tok = 0, masked_tok = 0, kept_seg = 0, veto_seg = 0;
  for (int g = threadIdx.x; g < S; g += kFinThreads) {
    const double* st = seg_stats + 4 * (size_t)g;
    const double n = st[0];
    bool keep = false, vetoed = false;
    float w = 1.f;
    if (n > 0) {
      const double mean = st[1] / n;
      w = (float)exp(mean);
      vetoed = st[2] < ln_veto;
      keep = (ln_lo <= mean) && (mean <= ln_hi) && !vetoed;
      if (keep_from_caller == 1) keep = seg_keep[g] != 0;            // the caller's decision stands
      else if (keep_from_caller == 2) keep = keep && seg_keep[g] != 0;  // caller's retention AND the MRS test
    }
    seg_w[g] = w;
    seg_keep[g] = keep ? 1 : 0;
    masked_tok += n;
    if (keep) { kept_tok += n; kept_seg += 1; }
    if (vetoed) veto_seg += 1;
  }
  kept_tok = block_sum(kept_tok, sh);
  masked_tok = block_sum(masked_tok, sh);
  kept_seg = block_sum(kept_seg, sh);
  veto_seg = block_sum(veto_seg, sh);
  double scale;
  if (norm == DRK_NORM_KEPT_TOKENS) scale = 1.0 / fmax(kept_tok, 1.0);
  else if (norm == DRK_NORM_ALL_MASKED_TOKENS) scale = 1.0 / fmax(masked_tok, 1.0);
  else scale = (double)explicit_scale;
  double part = 0.0;
  for (int g = threadIdx.x; g < S; g += kFinThreads) {
    double* st = seg_stats + 4 * (size_t)g;
    const double c = seg_keep[g] ? (double)seg_adv[g] * scale : 0.0;
    part += c * st[3];
    st[0] = c;  // per-segment coefficient, read by coeff_kernel
  }
  part = block_sum(part, sh);
  if (threadIdx.x == 0) {
    *loss = (float)(-part);
    counters[0] = (int64_t)kept_tok;
    counters[1] = (int64_t)masked_tok;
    counters[2] = (int64_t)kept_seg;
    counters[3] = (int64_t)veto_seg;
  }
}

__global__ void __launch_bounds__(kStatThreads)
coeff_kernel(const double* __restrict__ seg_stats, const uint8_t* __restrict__ mask,
             const int32_t* __restrict__ cu, int64_t T, float* __restrict__ coeff) {
  const int g = blockIdx.x;
  int64_t a = cu[g], b = cu[g + 1];
  if (a < 0 || b < a || b > T) return;
  const float c = (float)seg_stats[4 * (size_t)g];
  for (int64_t t = a + threadIdx.x; t < b; t += kStatThreads) coeff[t] = mask[t] ? c : 0.f;
}

__global__ void zero_scalars_kernel(float* loss, int64_t* counters) {
  *loss = 0.f;
  counters[0] = counters[1] = counters[2] = counters[3] = 0;
}

int launch_mrs(const MrsArgs& a, cudaStream_t st) {
  if (a.T > 0) DRK_CUDA_CHECK(cudaMemsetAsync(a.coeff, 0, sizeof(float) * (size_t)a.T, st));
  if (a.S == 0) {
    zero_scalars_kernel<<<1, 1, 0, st>>>(a.loss, a.counters);
    DRK_LAUNCHED();
    return DRK_OK;
  }
  seg_stats_kernel<<<a.S, kStatThreads, 0, st>>>(a.logp, a.rollout_logp, a.loss_mask, a.cu, a.T,
                                                  a.seg_stats, a.status);
  DRK_LAUNCHED();
  finalize_kernel<<<1, kFinThreads, 0, st>>>(a.seg_stats, a.seg_adv, a.S, a.ln_lo, a.ln_hi,
                                             a.ln_veto, a.norm, a.explicit_scale, a.keep_from_caller, a.seg_w,
                                             a.seg_keep, a.loss, a.counters);
  DRK_LAUNCHED();
  if (a.T > 0) {
    coeff_kernel<<<a.S, kStatThreads, 0, st>>>(a.seg_stats, a.loss_mask, a.cu, a.T, a.coeff);
    DRK_LAUNCHED();
  }
  return DRK_OK;
}

}  // namespace drk
