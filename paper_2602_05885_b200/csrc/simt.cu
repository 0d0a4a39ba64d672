// FFMA (CUDA-core) path of the fused LM-head loss: exact fp32 products and fp32 accumulation.
// It serves fp32 inputs, where tensor cores would round the operands, and doubles as an on-device
// cross-check of the tcgen05 path for bf16 inputs.
//
//   lmhead_fwd_kernel : 64x64 logit tiles, never stored; per row a running (max, sum-exp) carried
//                       over the block's vocabulary range, reduced across the 16 lanes that share a
//                       row with shuffles; the sampled token's logit is written by the one thread
//                       that owns it.
//   lse_merge_kernel  : merges the per-range (max, sum-exp, sum-exp-times-logit) partials into lse,
//                       logp and, on request, the token entropy (shared with the tcgen05 path).
//   lmhead_dl_kernel  : recomputes the tiles of one vocabulary chunk and stores
//                       dL = c_t (exp(s - lse_t) - onehot) in fp32.
//   gemm_kernel       : strided fp32 GEMM used for dW = dL^T hidden and dH += dL W.
#include "common.cuh"
#include <math_constants.h>

namespace drk {

constexpr int BM = 64, BN = 64, BK = 16, kThreads = 256;

// acc[i][j] += sum_k As[k][ty*4+i] * Bs[k][tx*4+j]
__device__ __forceinline__ void micro_kernel(const float (*As)[BM + 4], const float (*Bs)[BN + 4], int ty,
                                             int tx, float acc[4][4]) {
#pragma unroll
  for (int k = 0; k < BK; ++k) {
    const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
    const float4 b = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
    const float av[4] = {a.x, a.y, a.z, a.w};
    const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
  }
}

// Logit tile: rows [row0,row0+64) of hidden against rows [col0,col0+64) of W; both have the
// contraction index contiguous.  Out-of-range rows and columns read as zero.
template <typename TIn>
__device__ __forceinline__ void logit_tile(const TIn* __restrict__ hidden, const TIn* __restrict__ W,
                                           int64_t T, int H, int V, int64_t row0, int col0,
                                           float (*As)[BM + 4], float (*Bs)[BN + 4], float acc[4][4]) {
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const int lr = tid / 4, lk = (tid % 4) * 4;
  for (int k0 = 0; k0 < H; k0 += BK) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int k = k0 + lk + j;
      const int64_t r = row0 + lr;
      const int c = col0 + lr;
      As[lk + j][lr] = (r < T && k < H) ? to_f32(hidden[r * H + k]) : 0.f;
      Bs[lk + j][lr] = (c < V && k < H) ? to_f32(W[(int64_t)c * H + k]) : 0.f;
    }
    __syncthreads();
    micro_kernel(As, Bs, ty, tx, acc);
    __syncthreads();
  }
}

template <typename TIn>
__global__ void __launch_bounds__(kThreads)
lmhead_fwd_kernel(const TIn* __restrict__ hidden, const TIn* __restrict__ W, const int32_t* __restrict__ ids,
                  int64_t T, int H, int V, int tiles_per_split, float* __restrict__ part,
                  float* __restrict__ tgt, int id_off) {
  // part holds, per vocabulary range and row, {running max m, sum exp(s-m), sum exp(s-m)*s, unused}
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
  const int64_t row0 = (int64_t)blockIdx.x * BM;
  const int split = blockIdx.y;
  const int ntiles = (V + BN - 1) / BN;
  const int n_begin = split * tiles_per_split;
  const int n_end = min(ntiles, n_begin + tiles_per_split);
  float run_m[4], run_l[4], run_r[4];
  int target[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    run_m[i] = -CUDART_INF_F;
    run_l[i] = 0.f;
    run_r[i] = 0.f;
    const int64_t r = row0 + ty * 4 + i;
    target[i] = (r < T) ? local_id(ids[r], id_off, V) : -1;
  }
  for (int n = n_begin; n < n_end; ++n) {
    const int col0 = n * BN;
    float acc[4][4];
    logit_tile(hidden, W, T, H, V, row0, col0, As, Bs, acc);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float mx = -CUDART_INF_F;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = col0 + tx * 4 + j;
        if (c >= V) acc[i][j] = -CUDART_INF_F;
        mx = fmaxf(mx, acc[i][j]);
        if (c == target[i]) tgt[row0 + ty * 4 + i] = acc[i][j];
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(run_m[i], mx);
      float s = 0.f, sx = 0.f;
      if (m_new > -CUDART_INF_F) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float e = expf(acc[i][j] - m_new);
          s += e;
          sx += e * fmaxf(acc[i][j], -3.0e38f);   // masked columns (-inf) contribute 0, not 0 * inf
        }
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, o);
        sx += __shfl_xor_sync(0xffffffffu, sx, o);
      }
      const float resc = (run_m[i] > -CUDART_INF_F) ? expf(run_m[i] - m_new) : 0.f;
      run_l[i] = run_l[i] * resc + s;
      run_r[i] = run_r[i] * resc + sx;
      run_m[i] = m_new;
    }
  }
  if (tx == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t r = row0 + ty * 4 + i;
      if (r < T) {
        reinterpret_cast<float4*>(part)[(int64_t)split * T + r] = make_float4(run_m[i], run_l[i], run_r[i], 0.f);
      }
    }
  }
}

__global__ void lse_merge_kernel(const float* __restrict__ part, const float* __restrict__ tgt,
                                 const int32_t* __restrict__ ids, int64_t T, int V, int nsplit,
                                 float* __restrict__ logp, float* __restrict__ lse, float* __restrict__ entropy,
                                 uint32_t* __restrict__ status, const int32_t* __restrict__ rowmap,
                                 const int32_t* __restrict__ n_rows) {
  // r: row of the partials; t: the token it belongs to (they differ when the forward ran on gathered rows)
  const int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (r >= T) return;
  int64_t t = r;
  if (rowmap != nullptr) {
    if (r >= n_rows[0]) return;
    t = rowmap[r];
  }
  const float4* p4 = reinterpret_cast<const float4*>(part);
  float M = -CUDART_INF_F;
  for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p4[(int64_t)s * T + r].x);
  float L = 0.f, R = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float4 v = p4[(int64_t)s * T + r];
    if (v.x > -CUDART_INF_F) {
      const float w = expf(v.x - M);
      L += v.y * w;
      R += v.z * w;
    }
  }
  const float z = M + logf(L);
  const int id = ids[t];
  uint32_t bits = 0;
  float tg = 0.f;
  if (id >= 0 && id < V) tg = tgt[r]; else bits |= DRK_STATUS_BAD_ID;
  if (!isfinite(z)) bits |= DRK_STATUS_NONFINITE;
  lse[t] = z;
  logp[t] = tg - z;
  if (entropy != nullptr) entropy[t] = z - R / L;   // H = lse - sum_v p_v s_v
  if (bits) atomicOr(status, bits);
}

template <typename TIn>
__global__ void __launch_bounds__(kThreads)
lmhead_dl_kernel(const TIn* __restrict__ hidden, const TIn* __restrict__ W, const int32_t* __restrict__ ids,
                 const float* __restrict__ lse, const float* __restrict__ coeff, int64_t T, int H, int V,
                 int v0, int vc_this, int vc, float* __restrict__ dL, int id_off) {
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
  const int64_t row0 = (int64_t)blockIdx.x * BM;
  const int col0 = v0 + blockIdx.y * BN;
  float acc[4][4];
  logit_tile(hidden, W, T, H, V, row0, col0, As, Bs, acc);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t r = row0 + ty * 4 + i;
    if (r >= T) continue;
    const float c = coeff[r], z = lse[r];
    const int id = local_id(ids[r], id_off, V);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int v = col0 + tx * 4 + j;
      if (v - v0 >= vc_this) continue;
      float d = 0.f;
      if (c != 0.f) d = c * (expf(acc[i][j] - z) - (v == id ? 1.f : 0.f));
      dL[r * vc + (v - v0)] = d;
    }
  }
}

// C[m,n] (beta ? += : =) sum_k A[m*a_rs + k*a_cs] * B[k*b_rs + n*b_cs];  C row-major with ldc.
template <typename TB, typename TC>
__global__ void __launch_bounds__(kThreads)
gemm_kernel(const float* __restrict__ A, int64_t a_rs, int64_t a_cs, const TB* __restrict__ B, int64_t b_rs,
            int64_t b_cs, TC* __restrict__ C, int64_t ldc, int64_t M, int64_t N, int64_t K, int beta) {
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
  const int64_t m0 = (int64_t)blockIdx.x * BM, n0 = (int64_t)blockIdx.y * BN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int64_t k0 = 0; k0 < K; k0 += BK) {
    for (int e = tid; e < BM * BK; e += kThreads) {
      int mm, kk;
      if (a_cs == 1) { mm = e / BK; kk = e % BK; } else { kk = e / BM; mm = e % BM; }
      const int64_t m = m0 + mm, k = k0 + kk;
      As[kk][mm] = (m < M && k < K) ? A[m * a_rs + k * a_cs] : 0.f;
    }
    for (int e = tid; e < BN * BK; e += kThreads) {
      int nn, kk;
      if (b_rs == 1) { nn = e / BK; kk = e % BK; } else { kk = e / BN; nn = e % BN; }
      const int64_t n = n0 + nn, k = k0 + kk;
      Bs[kk][nn] = (n < N && k < K) ? to_f32(B[k * b_rs + n * b_cs]) : 0.f;
    }
    __syncthreads();
    micro_kernel(As, Bs, ty, tx, acc);
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = acc[i][j];
      if (beta) v += to_f32(C[m * ldc + n]);
      if constexpr (sizeof(TC) == 2) C[m * ldc + n] = __float2bfloat16(v); else C[m * ldc + n] = v;
    }
  }
}

// Statistics of one vocabulary range per row, from the range's partials: (max, sum-exp, sum-exp-times-logit)
// relative to that max, and the sampled token's logit if the token lies in the range, else 0.
__global__ void shard_stats_kernel(const float* __restrict__ part, const float* __restrict__ tgt,
                                   const int32_t* __restrict__ ids, int id_off, int64_t T, int V, int nsplit,
                                   float* __restrict__ stats, uint32_t* __restrict__ status) {
  const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (t >= T) return;
  const float4* p4 = reinterpret_cast<const float4*>(part);
  float M = -CUDART_INF_F;
  for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p4[(int64_t)s * T + t].x);
  float L = 0.f, R = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float4 v = p4[(int64_t)s * T + t];
    if (v.x > -CUDART_INF_F) {
      const float w = expf(v.x - M);
      L += v.y * w;
      R += v.z * w;
    }
  }
  const float tg = local_id(ids[t], id_off, V) >= 0 ? tgt[t] : 0.f;
  if (!isfinite(M) || !isfinite(L)) atomicOr(status, DRK_STATUS_NONFINITE);
  reinterpret_cast<float4*>(stats)[t] = make_float4(M, L, R, tg);
}

// All ranges' statistics [n_shards, T, 4] -> lse, logp, entropy of the whole vocabulary.
__global__ void shard_merge_kernel(const float* __restrict__ stats_all, int n_shards, const int32_t* __restrict__ ids,
                                   int64_t T, int V_total, float* __restrict__ logp, float* __restrict__ lse,
                                   float* __restrict__ entropy, uint32_t* __restrict__ status) {
  const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (t >= T) return;
  const float4* p4 = reinterpret_cast<const float4*>(stats_all);
  float M = -CUDART_INF_F;
  for (int s = 0; s < n_shards; ++s) M = fmaxf(M, p4[(int64_t)s * T + t].x);
  float L = 0.f, R = 0.f, tg = 0.f;
  for (int s = 0; s < n_shards; ++s) {
    const float4 v = p4[(int64_t)s * T + t];
    if (v.x > -CUDART_INF_F) {
      const float w = expf(v.x - M);
      L += v.y * w;
      R += v.z * w;
    }
    tg += v.w;   // zero from every range but the one that owns the token
  }
  const float z = M + logf(L);
  uint32_t bits = 0;
  const int id = ids[t];
  if (id < 0 || id >= V_total) { bits |= DRK_STATUS_BAD_ID; tg = 0.f; }
  if (!isfinite(z)) bits |= DRK_STATUS_NONFINITE;
  lse[t] = z;
  logp[t] = tg - z;
  if (entropy != nullptr) entropy[t] = z - R / L;
  if (bits) atomicOr(status, bits);
}

int launch_shard_stats(const float* part, const float* tgt, const int32_t* ids, int id_off, int64_t T, int V,
                       int nsplit, float* stats, uint32_t* status, cudaStream_t st) {
  shard_stats_kernel<<<(unsigned)ceil_div(T, 256), 256, 0, st>>>(part, tgt, ids, id_off, T, V, nsplit, stats, status);
  DRK_LAUNCHED();
  return DRK_OK;
}

int launch_shard_merge(const float* stats_all, int n_shards, const int32_t* ids, int64_t T, int V_total, float* logp,
                       float* lse, float* entropy, uint32_t* status, cudaStream_t st) {
  shard_merge_kernel<<<(unsigned)ceil_div(T, 256), 256, 0, st>>>(stats_all, n_shards, ids, T, V_total, logp, lse,
                                                                 entropy, status);
  DRK_LAUNCHED();
  return DRK_OK;
}

__global__ void f32_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t n) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += stride) dst[i] = __float2bfloat16(src[i]);
}

int launch_f32_to_bf16(const float* src, __nv_bfloat16* dst, size_t n, cudaStream_t st) {
  if (n == 0) return DRK_OK;
  const int64_t cap = (int64_t)sm_count() * 16;
  const int blocks = (int)((n + 1023) / 1024 < cap ? (n + 1023) / 1024 : cap);
  f32_to_bf16_kernel<<<blocks, 256, 0, st>>>(src, dst, n);
  DRK_LAUNCHED();
  return DRK_OK;
}

int launch_lse_merge(const float* part, const float* tgt, const int32_t* ids, int64_t T, int V, int nsplit,
                     float* logp, float* lse, float* entropy, uint32_t* status, const int32_t* rowmap,
                     const int32_t* n_rows, cudaStream_t st) {
  lse_merge_kernel<<<(unsigned)ceil_div(T, 256), 256, 0, st>>>(part, tgt, ids, T, V, nsplit, logp, lse, entropy,
                                                               status, rowmap, n_rows);
  DRK_LAUNCHED();
  return DRK_OK;
}

int simt_nsplit(int64_t T, int V) {
  // enough blocks to fill the GPU a few times over, at least two 64-wide tiles per range
  const int64_t row_tiles = ceil_div(T, BM);
  const int ntiles = (V + BN - 1) / BN;
  int64_t want = ceil_div((int64_t)sm_count() * 8, row_tiles > 0 ? row_tiles : 1);
  if (want < 1) want = 1;
  if (want > ntiles) want = ntiles;
  if (want > 64) want = 64;
  const int per = (int)ceil_div(ntiles, want);
  return (int)ceil_div(ntiles, per);
}

int launch_simt_fwd(const SimtFwdArgs& a, cudaStream_t st) {
  const int ntiles = (a.V + BN - 1) / BN;
  const int per = (int)ceil_div(ntiles, a.nsplit);
  dim3 grid((unsigned)ceil_div(a.T, BM), (unsigned)a.nsplit);
  if (a.in_dtype == DRK_F32)
    lmhead_fwd_kernel<float><<<grid, kThreads, 0, st>>>((const float*)a.hidden, (const float*)a.W, a.ids, a.T,
                                                        a.H, a.V, per, a.part, a.tgt, a.id_off);
  else
    lmhead_fwd_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>((const __nv_bfloat16*)a.hidden,
                                                                (const __nv_bfloat16*)a.W, a.ids, a.T, a.H,
                                                                a.V, per, a.part, a.tgt, a.id_off);
  DRK_LAUNCHED();
  if (a.stats != nullptr)
    return launch_shard_stats(a.part, a.tgt, a.ids, a.id_off, a.T, a.V, a.nsplit, a.stats, a.status, st);
  return launch_lse_merge(a.part, a.tgt, a.ids, a.T, a.V, a.nsplit, a.logp, a.lse, a.entropy, a.status, nullptr,
                          nullptr, st);
}

template <typename TIn>
static int simt_bwd_typed(const SimtBwdArgs& a, cudaStream_t st) {
  const TIn* hidden = (const TIn*)a.hidden;
  const TIn* W = (const TIn*)a.W;
  float* dh_acc = (a.dh_dtype == DRK_F32) ? (float*)a.dH : a.dH_acc;
  int chunk = 0;
  for (int v0 = 0; v0 < a.V; v0 += a.vc, ++chunk) {
    const int vc_this = min(a.vc, a.V - v0);
    dim3 g1((unsigned)ceil_div(a.T, BM), (unsigned)ceil_div(vc_this, BN));
    lmhead_dl_kernel<TIn><<<g1, kThreads, 0, st>>>(hidden, W, a.ids, a.lse, a.coeff, a.T, a.H, a.V, v0, vc_this,
                                                   a.vc, a.dL, a.id_off);
    DRK_LAUNCHED();
    // dW[v0:v0+vc_this, :] (+)= dL^T hidden      (M = v, N = h, K = t)
    dim3 g2((unsigned)ceil_div(vc_this, BM), (unsigned)ceil_div(a.H, BN));
    if (a.dw_dtype == DRK_F32)
      gemm_kernel<TIn, float><<<g2, kThreads, 0, st>>>(a.dL, 1, a.vc, hidden, a.H, 1, (float*)a.dW + (int64_t)v0 * a.H,
                                                       a.H, vc_this, a.H, a.T, a.dw_accumulate);
    else
      gemm_kernel<TIn, __nv_bfloat16><<<g2, kThreads, 0, st>>>(a.dL, 1, a.vc, hidden, a.H, 1,
                                                               (__nv_bfloat16*)a.dW + (int64_t)v0 * a.H, a.H,
                                                               vc_this, a.H, a.T, a.dw_accumulate);
    DRK_LAUNCHED();
    if (a.chunk_events != nullptr) DRK_CUDA_CHECK(cudaEventRecord(static_cast<cudaEvent_t>(a.chunk_events[chunk]), st));
    // dH (+)= dL W[v0:v0+vc_this, :]              (M = t, N = h, K = v)
    dim3 g3((unsigned)ceil_div(a.T, BM), (unsigned)ceil_div(a.H, BN));
    gemm_kernel<TIn, float><<<g3, kThreads, 0, st>>>(a.dL, a.vc, 1, W + (int64_t)v0 * a.H, a.H, 1, dh_acc, a.H, a.T,
                                                     a.H, vc_this, chunk > 0 ? 1 : 0);
    DRK_LAUNCHED();
  }
  if (a.dh_dtype == DRK_BF16)
    return launch_f32_to_bf16(dh_acc, (__nv_bfloat16*)a.dH, (size_t)a.T * a.H, st);
  return DRK_OK;
}

int launch_simt_bwd(const SimtBwdArgs& a, cudaStream_t st) {
  return a.in_dtype == DRK_F32 ? simt_bwd_typed<float>(a, st) : simt_bwd_typed<__nv_bfloat16>(a, st);
}

}  // namespace drk
