// Row compaction for the backward pass.
//
// A token whose coefficient c_t is zero (masked out, outside every segment, in a rejected sample, or
// with zero advantage) contributes nothing to dLogits, hence nothing to dW, and its dH row is zero.
// The backward therefore runs on the rows with c_t != 0 only: their indices are listed in order
// (rowmap), their hidden rows are gathered into a dense buffer that TMA can tile, and the count is
// left in device memory, from where the persistent GEMM kernels size their own work; the host
// never learns it and never synchronises.
//
//   count_kernel  : non-zeros per block of 1024 rows
//   offsets_kernel: exclusive scan of the block counts; total and total rounded up to 256
//   rowmap_kernel : stable compaction of row indices (ballot + popc), -1 behind the last one
//   gather_kernel : hidden_c[r,:] = hidden[rowmap[r],:], zero rows up to the rounded total
#include "common.cuh"

namespace drk {

constexpr int kBlk = 1024;

__global__ void __launch_bounds__(kBlk) count_kernel(const float* __restrict__ coeff, int64_t T,
                                                     int32_t* __restrict__ blk_cnt) {
  const int64_t t = (int64_t)blockIdx.x * kBlk + threadIdx.x;
  const bool nz = (t < T) && (coeff[t] != 0.f);
  const int c = __syncthreads_count(nz);
  if (threadIdx.x == 0) blk_cnt[blockIdx.x] = c;
}

__global__ void offsets_kernel(const int32_t* __restrict__ blk_cnt, int nblk, int32_t* __restrict__ blk_off,
                               int32_t* __restrict__ n_rows) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int acc = 0;
  for (int b = 0; b < nblk; ++b) {
    blk_off[b] = acc;
    acc += blk_cnt[b];
  }
  n_rows[0] = acc;
  n_rows[1] = (acc + 255) / 256 * 256;
}

__global__ void __launch_bounds__(kBlk) rowmap_kernel(const float* __restrict__ coeff, int64_t T,
                                                      const int32_t* __restrict__ blk_off,
                                                      const int32_t* __restrict__ n_rows, int64_t map_len,
                                                      int32_t* __restrict__ rowmap, uint32_t* __restrict__ status) {
  __shared__ int warp_cnt[kBlk / 32];
  const int64_t t = (int64_t)blockIdx.x * kBlk + threadIdx.x;
  const bool nz = (t < T) && (coeff[t] != 0.f);
  const unsigned m = __ballot_sync(0xffffffffu, nz);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) warp_cnt[w] = __popc(m);
  __syncthreads();
  int base = blk_off[blockIdx.x];
  for (int i = 0; i < w; ++i) base += warp_cnt[i];
  const int dst = base + __popc(m & ((1u << lane) - 1u));
  if (nz && DRK_IN_RANGE(dst >= 0 && dst < map_len, status)) rowmap[dst] = (int32_t)t;
  // entries behind the last compacted row (disjoint from the ones written above)
  const int total = n_rows[0];
  if (t >= total && t < map_len) rowmap[t] = -1;
}

__global__ void __launch_bounds__(256) gather_kernel(const __nv_bfloat16* __restrict__ hidden, int H,
                                                     const int32_t* __restrict__ rowmap,
                                                     const int32_t* __restrict__ n_rows,
                                                     __nv_bfloat16* __restrict__ hidden_c, int64_t T, int64_t map_len,
                                                     uint32_t* __restrict__ status) {
  int padded = n_rows[1];
  if (!DRK_IN_RANGE(padded >= 0 && padded <= map_len, status)) padded = 0;
  const int vec_per_row = H / 8;  // 16-byte vectors; H is a multiple of 8 on this path
  for (int r = blockIdx.x; r < padded; r += gridDim.x) {
    const int src = rowmap[r];
    uint4* dst = reinterpret_cast<uint4*>(hidden_c + (size_t)r * H);
    if (src >= 0 && DRK_IN_RANGE(src < T, status)) {
      const uint4* s = reinterpret_cast<const uint4*>(hidden + (size_t)src * H);
      for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x) dst[i] = s[i];
    } else {
      for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x) dst[i] = make_uint4(0, 0, 0, 0);
    }
  }
}

// dst[rowmap[r], :] = src[r, :] (fp32 -> fp32 or bf16), eight elements per thread and step.
__global__ void __launch_bounds__(256) scatter_rows_kernel(const float* __restrict__ src, int H,
                                                           const int32_t* __restrict__ rowmap,
                                                           const int32_t* __restrict__ n_rows, void* __restrict__ dst,
                                                           int dst_bf16, int64_t T, uint32_t* __restrict__ status) {
  const int cnt = n_rows[0];
  const int vec_per_row = H / 8;
  for (int r = blockIdx.x; r < cnt; r += gridDim.x) {
    const int t = rowmap[r];
    if (t < 0 || !DRK_IN_RANGE(t < T, status)) continue;
    const float4* s = reinterpret_cast<const float4*>(src + (size_t)r * H);
    for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x) {
      const float4 a = s[2 * i], b = s[2 * i + 1];
      if (dst_bf16) {
        __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y), p1 = __floats2bfloat162_rn(a.z, a.w);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x, b.y), p3 = __floats2bfloat162_rn(b.z, b.w);
        uint4 o;
        o.x = *reinterpret_cast<uint32_t*>(&p0); o.y = *reinterpret_cast<uint32_t*>(&p1);
        o.z = *reinterpret_cast<uint32_t*>(&p2); o.w = *reinterpret_cast<uint32_t*>(&p3);
        reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(dst) + (size_t)t * H)[i] = o;
      } else {
        float4* d = reinterpret_cast<float4*>(static_cast<float*>(dst) + (size_t)t * H);
        d[2 * i] = a;
        d[2 * i + 1] = b;
      }
    }
  }
}

int launch_scatter_rows(const float* src, int H, const int32_t* rowmap, const int32_t* n_rows, void* dst, bool dst_bf16,
                        int64_t T, uint32_t* status, cudaStream_t st) {
  scatter_rows_kernel<<<sm_count() * 8, 256, 0, st>>>(src, H, rowmap, n_rows, dst, dst_bf16 ? 1 : 0, T, status);
  DRK_LAUNCHED();
  return DRK_OK;
}

__global__ void __launch_bounds__(256) need_rows_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ cu,
                                                        int64_t T, float* __restrict__ need) {
  const int g = blockIdx.x;
  const int64_t a = cu[g], b = cu[g + 1];
  if (a < 0 || b < a || b > T) return;
  for (int64_t t = a + threadIdx.x; t < b; t += blockDim.x) need[t] = mask[t] ? 1.f : 0.f;
}

int launch_need_rows(const uint8_t* loss_mask, const int32_t* cu, int64_t T, int S, float* need, cudaStream_t st) {
  if (T == 0) return DRK_OK;
  DRK_CUDA_CHECK(cudaMemsetAsync(need, 0, sizeof(float) * (size_t)T, st));
  if (S == 0) return DRK_OK;
  need_rows_kernel<<<S, 256, 0, st>>>(loss_mask, cu, T, need);
  DRK_LAUNCHED();
  return DRK_OK;
}

int64_t compact_map_len(int64_t T) { return (T + 255) / 256 * 256 + 256; }
int compact_blocks(int64_t T) { return (int)((compact_map_len(T) + kBlk - 1) / kBlk); }

int launch_compact(const CompactArgs& a, cudaStream_t st) {
  const int nblk = compact_blocks(a.T);
  const int64_t map_len = compact_map_len(a.T);
  count_kernel<<<nblk, kBlk, 0, st>>>(a.coeff, a.T, a.blk_cnt);
  DRK_LAUNCHED();
  offsets_kernel<<<1, 32, 0, st>>>(a.blk_cnt, nblk, a.blk_off, a.n_rows);
  DRK_LAUNCHED();
  rowmap_kernel<<<nblk, kBlk, 0, st>>>(a.coeff, a.T, a.blk_off, a.n_rows, map_len, a.rowmap, a.status);
  DRK_LAUNCHED();
  gather_kernel<<<sm_count() * 8, 256, 0, st>>>(a.hidden, a.H, a.rowmap, a.n_rows, a.hidden_c, a.T, map_len, a.status);
  DRK_LAUNCHED();
  return DRK_OK;
}

}  // namespace drk
