// Reward front-end: per-turn reward (Sec. 4.2, Eq. 1), profiling-based reward and profiling-based
// rejection sampling (Sec. 5.2; hard-threshold variant of App. D).
//
// One thread per (rollout, turn) sample; a few thousand scalars, latency-bound.  The retention draw
// is Philox-4x32-10 keyed by the caller's seed with counter (sample index, offset), so a run is
// reproducible and independent of launch shape.
#include "common.cuh"

namespace drk {

__device__ __forceinline__ void philox_round(uint32_t (&c)[4], uint32_t k0, uint32_t k1) {
  const uint32_t hi0 = __umulhi(0xD2511F53u, c[0]), lo0 = 0xD2511F53u * c[0];
  const uint32_t hi1 = __umulhi(0xCD9E8D57u, c[2]), lo1 = 0xCD9E8D57u * c[2];
  const uint32_t n0 = hi1 ^ c[1] ^ k0, n2 = hi0 ^ c[3] ^ k1;
  c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
}

// First output word of Philox-4x32 with 10 rounds.
__device__ __forceinline__ uint32_t philox4x32_10_x0(uint64_t index, uint64_t offset, uint64_t seed) {
  uint32_t c[4] = {(uint32_t)index, (uint32_t)(index >> 32), (uint32_t)offset, (uint32_t)(offset >> 32)};
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    philox_round(c, k0, k1);
  }
  return c[0];
}

__global__ void reward_kernel(const uint8_t* __restrict__ correct, const float* __restrict__ t_ref,
                              const float* __restrict__ t_kernel, const float* __restrict__ pr, int64_t n,
                              float clip, int use_pr, int prs_mode, float tau, float s, uint64_t seed,
                              uint64_t offset, float* __restrict__ reward, uint8_t* __restrict__ retain) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  const bool c = correct[i] != 0;
  float r = 0.f;
  if (c) {
    r = 1.f + fminf(__fdiv_rn(t_ref[i], t_kernel[i]), clip);
    if (use_pr) r += pr[i];
  }
  reward[i] = r;
  if (retain != nullptr) {
    bool keep = true;
    if (prs_mode == 2) {
      keep = pr[i] >= tau;
    } else if (prs_mode == 1) {
      // p = clip((PR - tau) / s, 0, 1) in fp32 without contraction; u = top 24 bits * 2^-24
      const float p = fminf(fmaxf(__fdiv_rn(__fsub_rn(pr[i], tau), s), 0.f), 1.f);
      const float u = (float)(philox4x32_10_x0((uint64_t)i, offset, seed) >> 8) * (1.0f / 16777216.0f);
      keep = u < p;
    }
    retain[i] = keep ? 1 : 0;
  }
}

int launch_reward(const uint8_t* correct, const float* t_ref, const float* t_kernel, const float* pr, int64_t n,
                  const drk_reward_params& p, float* reward, uint8_t* retain, cudaStream_t st) {
  if (n == 0) return DRK_OK;
  reward_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(correct, t_ref, t_kernel, pr, n, p.speedup_clip,
                                                            p.use_pr, p.prs_mode, p.prs_tau, p.prs_s, p.seed,
                                                            p.offset, reward, retain);
  DRK_LAUNCHED();
  return DRK_OK;
}

}  // namespace drk

using namespace drk;

extern "C" void drk_reward_params_default(drk_reward_params* p) {
  if (!p) return;
  p->speedup_clip = 3.0f;
  p->use_pr = 0;
  p->prs_mode = DRK_PRS_OFF;
  p->prs_tau = 0.3f;
  p->prs_s = 0.1f;
  p->seed = 0;
  p->offset = 0;
}

extern "C" int drk_reward(const uint8_t* correct, const float* t_ref, const float* t_kernel, const float* pr,
                          int64_t n, const drk_reward_params* pp, float* reward, uint8_t* retain, void* stream) {
  g_launches = 0;
  drk_reward_params p;
  if (pp) p = *pp; else drk_reward_params_default(&p);
  if (n < 0 || n > ((int64_t)1 << 31)) return DRK_ERR_INVALID_ARG;
  if (p.prs_mode < DRK_PRS_OFF || p.prs_mode > DRK_PRS_HARD) return DRK_ERR_INVALID_ARG;
  if (!(p.speedup_clip > 0.f) || (p.prs_mode == DRK_PRS_SOFT && !(p.prs_s > 0.f))) return DRK_ERR_INVALID_ARG;
  if (n == 0) return DRK_OK;
  if (!correct || !t_ref || !t_kernel || !reward) return DRK_ERR_INVALID_ARG;
  if ((p.use_pr || p.prs_mode != DRK_PRS_OFF) && !pr) return DRK_ERR_INVALID_ARG;
  if (p.prs_mode != DRK_PRS_OFF && !retain) return DRK_ERR_INVALID_ARG;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return DRK_ERR_CUDA;
  if (major != 10) return DRK_ERR_ARCH;
  const int rc = launch_reward(correct, t_ref, t_kernel, pr, n, p, reward, retain, static_cast<cudaStream_t>(stream));
  if (rc != DRK_OK) g_launches = 0;
  return rc;
}
