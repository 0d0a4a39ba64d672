// Stability diagnostics over one micro-batch: the quantities the paper monitors to spot training /
// inference mismatch (Sec. 5.1, App. B): mean token entropy, perplexity under the trainer and under
// the rollout engine, mean and largest log-ratio, gradient norms.
//
// The entropy itself comes out of the forward kernels (it needs the logits); everything here is a
// pass over T floats, plus one streaming pass over dH and dW when their norms are asked for.
// Sums are accumulated with fp64 atomics, so the last digits can differ from run to run.
#include "common.cuh"

namespace drk {

constexpr int kDiagThreads = 256;

__device__ __forceinline__ double warp_sum_d(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// acc: [0] n, [1] sum entropy, [2] sum logp, [3] sum rollout_logp, [4] sum delta, [5] max |delta| (as bits)
__global__ void __launch_bounds__(kDiagThreads)
diag_tokens_kernel(const float* __restrict__ logp, const float* __restrict__ rollout_logp,
                   const float* __restrict__ entropy, const uint8_t* __restrict__ mask,
                   const int32_t* __restrict__ cu, int64_t T, double* __restrict__ acc) {
  const int g = blockIdx.x;
  int64_t a = cu[g], b = cu[g + 1];
  if (a < 0 || b < a || b > T) return;
  double n = 0, se = 0, sl = 0, sr = 0, sd = 0, mx = 0;
  for (int64_t t = a + threadIdx.x; t < b; t += kDiagThreads) {
    if (!mask[t]) continue;
    const double lp = logp[t], rl = rollout_logp[t];
    n += 1;
    if (entropy != nullptr) se += entropy[t];
    sl += lp;
    sr += rl;
    sd += lp - rl;
    mx = fmax(mx, fabs(lp - rl));
  }
  n = warp_sum_d(n); se = warp_sum_d(se); sl = warp_sum_d(sl); sr = warp_sum_d(sr); sd = warp_sum_d(sd);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0 && n > 0) {
    atomicAdd(acc + 0, n);
    atomicAdd(acc + 1, se);
    atomicAdd(acc + 2, sl);
    atomicAdd(acc + 3, sr);
    atomicAdd(acc + 4, sd);
    // non-negative doubles order like their bit patterns
    atomicMax(reinterpret_cast<unsigned long long*>(acc + 5), (unsigned long long)__double_as_longlong(mx));
  }
}

template <typename T>
__global__ void __launch_bounds__(kDiagThreads) sumsq_kernel(const T* __restrict__ x, size_t n, double* __restrict__ out) {
  double s = 0;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += stride) {
    const double v = (double)to_f32(x[i]);
    s += v * v;
  }
  s = warp_sum_d(s);
  __shared__ double sh[kDiagThreads / 32];
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double r = 0;
    for (int w = 0; w < kDiagThreads / 32; ++w) r += sh[w];
    atomicAdd(out, r);
  }
}

// acc (sums) -> out (means, perplexities, norms), in place
__global__ void diag_finalize_kernel(double* __restrict__ d) {
  const double n = d[0];
  const double se = d[1], sl = d[2], sr = d[3], sd = d[4], mx = d[5], qh = d[6], qw = d[7];
  d[1] = n > 0 ? se / n : 0.0;
  d[2] = n > 0 ? exp(-sl / n) : 1.0;
  d[3] = n > 0 ? exp(-sr / n) : 1.0;
  d[4] = n > 0 ? sd / n : 0.0;
  d[5] = mx;
  d[6] = sqrt(qh);
  d[7] = sqrt(qw);
}

static int launch_sumsq(const void* x, int dtype, size_t n, double* out, cudaStream_t st) {
  if (x == nullptr || n == 0) return DRK_OK;
  const int64_t cap = (int64_t)sm_count() * 8;
  const int blocks = (int)((n + 4095) / 4096 < cap ? (n + 4095) / 4096 : cap);
  if (dtype == DRK_BF16) sumsq_kernel<__nv_bfloat16><<<blocks, kDiagThreads, 0, st>>>((const __nv_bfloat16*)x, n, out);
  else sumsq_kernel<float><<<blocks, kDiagThreads, 0, st>>>((const float*)x, n, out);
  DRK_LAUNCHED();
  return DRK_OK;
}

}  // namespace drk

using namespace drk;

extern "C" int drk_pg_diagnostics(const float* logp, const float* rollout_logp, const float* entropy,
                                  const uint8_t* loss_mask, const int32_t* cu_seqlens, int64_t T, int32_t S,
                                  const void* dH, int32_t dh_dtype, const void* dW, int32_t dw_dtype, int32_t H,
                                  int32_t V, double* out, void* stream) {
  g_launches = 0;
  if (T < 0 || S < 0 || H < 0 || V < 0 || !out) return DRK_ERR_INVALID_ARG;
  if ((dH && dh_dtype != DRK_F32 && dh_dtype != DRK_BF16) || (dW && dw_dtype != DRK_F32 && dw_dtype != DRK_BF16))
    return DRK_ERR_INVALID_ARG;
  if (S > 0 && T > 0 && (!logp || !rollout_logp || !loss_mask || !cu_seqlens)) return DRK_ERR_INVALID_ARG;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return DRK_ERR_CUDA;
  if (major != 10) return DRK_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto fail = [&](int code) { g_launches = 0; return code; };
  if (cudaMemsetAsync(out, 0, 8 * sizeof(double), st) != cudaSuccess) return fail(DRK_ERR_CUDA);
  if (S > 0 && T > 0) {
    diag_tokens_kernel<<<S, kDiagThreads, 0, st>>>(logp, rollout_logp, entropy, loss_mask, cu_seqlens, T, out);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return fail(DRK_ERR_CUDA);
  }
  int rc = launch_sumsq(dH, dh_dtype, (size_t)T * (size_t)H, out + 6, st);
  if (rc != DRK_OK) return fail(rc);
  rc = launch_sumsq(dW, dw_dtype, (size_t)V * (size_t)H, out + 7, st);
  if (rc != DRK_OK) return fail(rc);
  diag_finalize_kernel<<<1, 1, 0, st>>>(out);
  ++g_launches;
  if (cudaGetLastError() != cudaSuccess) return fail(DRK_ERR_CUDA);
  return DRK_OK;
}
