// tcgen05 path of the fused LM-head loss (bf16 operands, fp32 accumulation in tensor memory).
//
// One persistent, warp-specialised GEMM kernel, instantiated for the four contractions of the path:
//
//   FWD : S = hidden W^T tile by tile; epilogue keeps a running (max, sum-exp, sum-exp*logit) per row over
//         the unit's vocabulary range and picks out the sampled token's logit.  Logits never leave the SM.
//   DL  : the same tiles for one vocabulary chunk; epilogue forms
//         dL = c_t (exp(s - lse_t) - onehot) as bf16 into the chunk buffer [T, vc].
//   DW  : dW[chunk] (+)= dL^T hidden        (both operands have M/N contiguous: MN-major)
//   DH  : dH_acc (+)= dL W[chunk]           (A K-major, B MN-major; fp32 accumulator over the compacted rows)
//
// Tile 128 x 256 x 64 per CTA (256 x 256 per CTA pair with cta_group::2), one CTA per SM, 192 threads:
//   warp 0    : TMA producer (one lane): 128B-swizzled operand tiles into a ring of stages; in the even
//               CTA it also draws the block's next work unit from a device-side counter and announces it
//   warp 1    : tensor-memory allocation; one lane issues tcgen05.mma (K = 16 each) into one of two
//               256-column fp32 accumulators and commits to mbarriers
//   warps 2-5 : epilogue; warp w reads tensor-memory lanes 32*(w%4)..+31, one accumulator row per
//               thread, 32 columns per tcgen05.ld, while the MMA warp fills the other accumulator.
//               DL / DW / DH stage their output in swizzled shared memory and let the TMA unit store it
//               (or add it, at the memory side, to what is there).
// Every mbarrier wait is bounded; on expiry the block raises DRK_STATUS_TIMEOUT, drains its
// in-flight copies and MMAs, frees tensor memory and returns.
#include "common.cuh"
#include "umma.cuh"
#include "umma_plan.cuh"
#include <atomic>
#include <math_constants.h>
#include <mutex>
#include <unordered_map>

namespace drk {

namespace {

constexpr int TM = 128, TN = 256, TK = 64;
constexpr int A_BYTES = TM * TK * 2;      // 16 KiB: 128 rows of A per CTA
// 64-deep k-blocks per pipeline stage of a CTA pair.  Two (three 64 KiB stages, eight MMAs per
// tcgen05.commit) measured 4 % faster end to end than one (six 32 KiB stages, four MMAs per commit).
// The backward's row padding (256 rows) covers at most four k-blocks per stage.
#ifndef DRK_STAGE_SUBS
#define DRK_STAGE_SUBS 2
#endif
static_assert(DRK_STAGE_SUBS == 1 || DRK_STAGE_SUBS == 2 || DRK_STAGE_SUBS == 4, "stage depth must divide the 256-row padding");
#ifndef DRK_RING_KB
#define DRK_RING_KB 192
#endif
constexpr int RING_BYTES = DRK_RING_KB * 1024;  // operand ring: 4 stages of 48 KiB, or 6 of 32 KiB for a CTA pair
constexpr int MAX_STAGES = 8;
constexpr int SUB_BYTES = 64 * TK * 2;    // one 64-wide MN-major box: 64 k-rows x 128 B
constexpr int NUM_THREADS = 192;
constexpr int SCHED_SLOTS = 4;            // work units announced ahead of their use (dynamic schedule)
constexpr int NUM_BARS = 2 * MAX_STAGES + 5 + 2 * SCHED_SLOTS;
// Output staging for the TMA stores of the backward's epilogues: per epilogue warp two boxes of 32 rows x 128
// bytes (128B-swizzled), so that a box can be filled while the TMA unit still reads the previous one.
constexpr int OUT_BOX_BYTES = 32 * 128;
constexpr int OUT_STAGE_BYTES = 4 * 2 * OUT_BOX_BYTES;
constexpr int SMEM_BYTES = RING_BYTES + OUT_STAGE_BYTES + 1024 /*alignment slack*/ + NUM_BARS * 8 + 16 + 4 * SCHED_SLOTS;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory per block");
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;  // 2 s: far above any legitimate wait
constexpr uint64_t DRAIN_LIMIT_NS = 20000000ull;   // 20 ms per outstanding copy when giving up
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

enum Mode { FWD = 0, DL = 1, DW = 2, DH = 3 };

struct UmmaParams {
  int m_tiles, n_tiles, k_blocks, group_m, nj, tiles_per_unit, num_units;
  // Order of the work units.  group_n == 0: groups of group_m row tiles, within a group the column index
  // is the slow one (the group's A panels stay in L2 while it sweeps the columns).  group_n > 0: groups of
  // group_n column units, within a group the row tile is the slow index (the group's B panels stay in L2
  // while the rows stream past).
  int group_n;
  int64_t rows;  // valid extent of the tile-row index (T, or the chunk's width for DW)
  int cols;      // valid extent of the tile-column index (V, the chunk's width, or H)
  int v0;        // first vocabulary column of the chunk (0 for FWD)
  int id_off;    // W holds columns [id_off, id_off + width) of a larger vocabulary: ids are taken relative to it
  int id_width;  // number of columns W holds
  int64_t T;
  const int32_t* ids;
  const float* lse;
  const float* coeff;
  float* part;
  float* tgt;
  int want_entropy;  // FWD: also carry sum exp(s-m)*s per row
  __nv_bfloat16* dL;
  int vc;
  void* C;
  const void* C_in;
  int64_t ldc;
  int beta, out_bf16, in_bf16;
  // How the epilogue of DL / DW / DH writes its tile: 0 = from registers (16-byte stores per thread, with a
  // read-modify-write when beta is set); 1 = staged in shared memory and stored by the TMA unit through the
  // output tensor map; 2 = the same with an element-wise add at the memory side (fp32 accumulation without
  // the SM ever loading the old values).
  int out_tma;
  uint32_t* status;
  // Compacted backward: the row dimension (M for DL and DH, K for DW) runs over the rows listed in
  // rowmap; their number is n_rows[0] (n_rows[1] = rounded up to 256), known on the device only.
  const int32_t* rowmap;
  const int32_t* n_rows;
  // Dynamic schedule: a zeroed counter from which the blocks (CTA pairs) draw their next work unit as they
  // finish one, so that the units in flight are always consecutive ones.  Null: unit u goes to block
  // u mod (number of blocks).
  int32_t* sched;
};

struct Unit {
  int m, j, n_begin, n_end;
};

__device__ __forceinline__ Unit decode_unit(const UmmaParams& p, int m_tiles, int u) {
  if (p.group_n > 0) {
    const int per_group = m_tiles * p.group_n;      // every group but the last holds group_n column units
    const int g = u / per_group;
    const int rem = u - g * per_group;
    const int gn = min(p.group_n, p.nj - g * p.group_n);
    Unit r;
    r.m = rem / gn;
    r.j = g * p.group_n + rem % gn;
    r.n_begin = r.j * p.tiles_per_unit;
    r.n_end = min(p.n_tiles, r.n_begin + p.tiles_per_unit);
    return r;
  }
  const int per_group = p.group_m * p.nj;
  const int g = u / per_group;
  const int rem = u - g * per_group;
  const int gm = min(p.group_m, m_tiles - g * p.group_m);
  Unit r;
  r.j = rem / gm;
  r.m = g * p.group_m + rem % gm;
  r.n_begin = r.j * p.tiles_per_unit;
  r.n_end = min(p.n_tiles, r.n_begin + p.tiles_per_unit);
  return r;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t raw_bits(float v) { return __float_as_uint(v); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Warp-collective bounded wait: all 32 lanes poll, and leave together.
template <bool CLUSTER_ACQUIRE = false>
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort, int lane) {
  uint64_t t0 = 0;
  uint32_t polls = 0;
#pragma unroll 1
  for (;;) {
    const bool done = CLUSTER_ACQUIRE ? ptx::mbar_try_wait_cluster(bar, parity) : ptx::mbar_try_wait(bar, parity);
    if (__all_sync(0xffffffffu, done)) return true;
    if ((++polls & 0x3ffu) == 0) {
      if (t0 == 0) t0 = ptx::globaltimer_ns();
      const bool give_up = (*abort != 0) || (ptx::globaltimer_ns() - t0 > WAIT_LIMIT_NS);
      if (__any_sync(0xffffffffu, give_up)) {
        if (lane == 0) *abort = 1;
        return false;
      }
    }
  }
}

// Store 32 consecutive fp32 results of one row, optionally added to what is there, as fp32 or bf16.
__device__ __forceinline__ void store_row_chunk(const UmmaParams& p, int64_t row, int col, float (&x)[32]) {
  const int64_t off = row * p.ldc + col;
  const int nvalid = min(32, p.cols - col);
  if (nvalid == 32) {
    if (p.beta) {
      if (p.in_bf16) {
        const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.C_in) + off);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 w = src[q];
          const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            x[q * 8 + e * 2 + 0] += __uint_as_float(ws[e] << 16);
            x[q * 8 + e * 2 + 1] += __uint_as_float(ws[e] & 0xffff0000u);
          }
        }
      } else {
        const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.C_in) + off);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float4 w = src[q];
          x[q * 4 + 0] += w.x; x[q * 4 + 1] += w.y; x[q * 4 + 2] += w.z; x[q * 4 + 3] += w.w;
        }
      }
    }
    if (p.out_bf16) {
      uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.C) + off);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        dst[q] = make_uint4(pack_bf16(x[q * 8 + 0], x[q * 8 + 1]), pack_bf16(x[q * 8 + 2], x[q * 8 + 3]),
                            pack_bf16(x[q * 8 + 4], x[q * 8 + 5]), pack_bf16(x[q * 8 + 6], x[q * 8 + 7]));
    } else {
      float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.C) + off);
#pragma unroll
      for (int q = 0; q < 8; ++q) dst[q] = make_float4(x[q * 4 + 0], x[q * 4 + 1], x[q * 4 + 2], x[q * 4 + 3]);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      if (j < nvalid) {
        float v = x[j];
        if (p.beta)
          v += p.in_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.C_in)[off + j])
                         : reinterpret_cast<const float*>(p.C_in)[off + j];
        if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.C)[off + j] = __float2bfloat16(v);
        else reinterpret_cast<float*>(p.C)[off + j] = v;
      }
    }
  }
}

// CTAS = 1: one CTA per 128x256 tile.  CTAS = 2: a pair of CTAs (cluster of two) shares a 256x256
// tile through tcgen05 cta_group::2: each CTA loads its 128 rows of A and its 128 of B's 256 rows,
// the even CTA issues the MMAs for both, and each CTA drains its own 128 accumulator rows.
template <int MODE, int CTAS>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmC, const UmmaParams p) {
  constexpr bool A_MN = (MODE == DW);
  constexpr bool B_MN = (MODE == DW || MODE == DH);
  constexpr uint32_t IDESC = ptx::make_idesc_bf16(TM * CTAS, TN, A_MN ? 1 : 0, B_MN ? 1 : 0);
  constexpr int BN_CTA = TN / CTAS;                 // rows of B this CTA loads
  constexpr int B_BYTES_CTA = BN_CTA * TK * 2;
  constexpr int SUBS = (CTAS == 2) ? DRK_STAGE_SUBS : 1;  // 64-deep k-blocks per pipeline stage
  constexpr int SUB = A_BYTES + B_BYTES_CTA;        // bytes of one k-block (A rows + B rows of this CTA)
  constexpr int STAGE = SUBS * SUB;                 // bytes per stage in this CTA
  constexpr int NSTAGE = RING_BYTES / STAGE;
  constexpr uint32_t TX_BYTES = STAGE * CTAS;       // both CTAs' loads are credited to one barrier

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = ptx::smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const uint32_t smem_base = raw_addr + pad;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + RING_BYTES + OUT_STAGE_BYTES);
  const uint32_t bar_base = smem_base + RING_BYTES + OUT_STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + 2 + a); };
  const uint32_t done_bar = bar_base + 8u * (2 * MAX_STAGES + 4);
  auto ufull_bar = [&](int s) { return bar_base + 8u * (2 * MAX_STAGES + 5 + s); };
  auto uempty_bar = [&](int s) { return bar_base + 8u * (2 * MAX_STAGES + 5 + SCHED_SLOTS + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* unit_slot = reinterpret_cast<volatile int*>(tmem_slot + 4);   // [SCHED_SLOTS]
  const uint32_t unit_slot_addr = ptx::smem_u32(tmem_slot + 4);

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const int cta_rank = (CTAS == 2) ? (int)ptx::cluster_ctarank() : 0;
  const bool leader = (cta_rank == 0);
  const int first_unit = blockIdx.x / CTAS, unit_stride = gridDim.x / CTAS;

  // Work extents: fixed by the host, or derived from the device-side count of compacted rows.
  int m_tiles = p.m_tiles, k_blocks = p.k_blocks;
  int64_t rows = p.rows;
  if (p.n_rows != nullptr) {
    const int cnt = p.n_rows[0];
    if constexpr (MODE == FWD || MODE == DL || MODE == DH) {
      m_tiles = (cnt + TM * CTAS - 1) / (TM * CTAS);
      rows = p.n_rows[1];
    }
    if constexpr (MODE == DW) k_blocks = (cnt + TK - 1) / TK;
  }
  int num_units = m_tiles * p.nj;
  // checked build: the device-side row count must fit what the host sized the buffers for
  if (!DRK_IN_RANGE(m_tiles >= 0 && m_tiles <= p.m_tiles && k_blocks >= 0 && k_blocks <= p.k_blocks, p.status))
    num_units = 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), 4 * CTAS);
    }
    ptx::mbar_init(done_bar, 1);
    for (int q = 0; q < SCHED_SLOTS; ++q) {
      ptx::mbar_init(ufull_bar(q), 1);
      // readers of a published unit: MMA thread and four epilogue warps in the even CTA; the producer
      // thread and four epilogue warps in the odd one.  All of them release the slot in the even CTA.
      ptx::mbar_init(uempty_bar(q), 5 * CTAS);
    }
    *abort = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    if constexpr (CTAS == 2) {
      ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), 512);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before();
  if constexpr (CTAS == 2) ptx::cluster_sync(); else __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // ---- work feed -------------------------------------------------------------------------------
  // Static: the n-th unit of this block is first_unit + n * unit_stride.  Dynamic (p.sched): the even CTA's
  // producer thread draws unit numbers from the global counter and announces the n-th one in slot
  // n % SCHED_SLOTS of both CTAs' shared memory; every other role reads it there and releases the slot.
  const bool dynamic = (p.sched != nullptr);
  auto static_unit = [&](uint32_t n) {
    const int64_t u = (int64_t)first_unit + (int64_t)n * unit_stride;
    return u < num_units ? (int)u : -1;
  };
  // one thread: wait for the n-th announcement, read it, release the slot; -2 on a timed-out wait
  auto take_unit = [&](uint32_t n) -> int {
    if (!dynamic) return static_unit(n);
    const int slot = n % SCHED_SLOTS;
    if (!ptx::mbar_wait<true>(ufull_bar(slot), (n / SCHED_SLOTS) & 1u, abort, WAIT_LIMIT_NS)) return -2;
    const int u = unit_slot[slot];
    if (CTAS == 2 && !leader) ptx::mbar_arrive_remote(uempty_bar(slot), 0);
    else ptx::mbar_arrive(uempty_bar(slot));
    return u;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmA);
      ptx::prefetch_tensormap(&tmB);
      uint32_t it = 0;
      bool ok = true;
      auto load = [&](uint32_t dst, const void* map, uint32_t bar, int x, int y) {
        if constexpr (CTAS == 2) ptx::tma_load_2d_pair(dst, map, bar, x, y);
        else ptx::tma_load_2d(dst, map, bar, x, y);
      };
      // Even CTA, dynamic schedule: announce the n-th unit of this block to every other role of both CTAs.
      auto announce = [&](uint32_t n, int u) -> bool {
        const int slot = n % SCHED_SLOTS;
        if (!ptx::mbar_wait(uempty_bar(slot), ((n / SCHED_SLOTS) & 1u) ^ 1u, abort, WAIT_LIMIT_NS)) return false;
        unit_slot[slot] = u;
        if constexpr (CTAS == 2) {
          ptx::st_shared_remote(unit_slot_addr + 4u * slot, 1, (uint32_t)u);
          ptx::mbar_arrive_remote(ufull_bar(slot), 1);   // release at cluster scope: orders the store above
        }
        ptx::mbar_arrive(ufull_bar(slot));
        return true;
      };
      auto drawn = [&](int v) { return (int64_t)v + unit_stride < num_units ? v + unit_stride : -1; };
      const bool feeder = dynamic && leader;
      uint32_t seq = 0;
      int u = -1, u_next = -1;
      if (feeder) {
        // the first unit is the block's own index; the counter hands out the units behind the first round.
        // Units are announced one ahead, so that the other CTA's producer never waits for this one's loads.
        u = static_unit(0);
        if (u >= 0) u_next = drawn(atomicAdd(p.sched, 1));
        ok = announce(0, u);
      } else {
        u = take_unit(0);
      }
      while (u >= 0 && ok) {
        int pending = -1;
        bool drew = false;
        if (feeder) {
          if (!announce(seq + 1, u_next)) { ok = false; break; }
          if (u_next >= 0) { pending = atomicAdd(p.sched, 1); drew = true; }   // consumed after this unit's loads
        }
        const Unit un = decode_unit(p, m_tiles, u);
        const int a_row = (un.m * CTAS + cta_rank) * TM;   // first A row (M index) of this CTA
        for (int n = un.n_begin; n < un.n_end && ok; ++n) {
          const int b_row = n * TN + cta_rank * BN_CTA;     // first B row (N index) of this CTA
          for (int kb0 = 0; kb0 < k_blocks; kb0 += SUBS) {
            const int s = it % NSTAGE;
            const uint32_t ph = (it / NSTAGE) & 1u;
            if (!ptx::mbar_wait(empty_bar(s), ph ^ 1u, abort, WAIT_LIMIT_NS)) { ok = false; break; }
            if (leader) ptx::mbar_arrive_expect_tx(full_bar(s), TX_BYTES);
#pragma unroll
            for (int sub = 0; sub < SUBS; ++sub) {
              // a k-block past the end of K lies outside the tensor and is filled with zeros
              const int kb = kb0 + sub;
              const uint32_t sa = smem_base + s * STAGE + sub * SUB, sb = sa + A_BYTES;
              if constexpr (MODE == FWD || MODE == DL) {
                load(sa, &tmA, full_bar(s), kb * TK, a_row);
                load(sb, &tmB, full_bar(s), kb * TK, p.v0 + b_row);
              } else if constexpr (MODE == DW) {
#pragma unroll
                for (int j = 0; j < TM / 64; ++j) load(sa + j * SUB_BYTES, &tmA, full_bar(s), a_row + 64 * j, kb * TK);
#pragma unroll
                for (int j = 0; j < BN_CTA / 64; ++j) load(sb + j * SUB_BYTES, &tmB, full_bar(s), b_row + 64 * j, kb * TK);
              } else {  // DH
                load(sa, &tmA, full_bar(s), kb * TK, a_row);
#pragma unroll
                for (int j = 0; j < BN_CTA / 64; ++j)
                  load(sb + j * SUB_BYTES, &tmB, full_bar(s), b_row + 64 * j, p.v0 + kb * TK);
              }
            }
            ++it;
          }
        }
        ++seq;
        if (feeder) { u = u_next; u_next = drew ? drawn(pending) : -1; }
        else u = take_unit(seq);
      }
      if (u == -2) ok = false;
      if (!ok && leader) {
        // wait (bounded) for the copies still in flight before the block leaves (a pair's loads are
        // all credited to the even CTA's barriers; the odd CTA waits for its peer at the cluster barrier)
        const uint32_t first = it > (uint32_t)NSTAGE ? it - NSTAGE : 0;
        for (uint32_t j = first; j < it; ++j)
          ptx::mbar_wait(full_bar(j % NSTAGE), (j / NSTAGE) & 1u, nullptr, DRAIN_LIMIT_NS);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA of a pair)
    if (lane == 0 && leader) {
      uint32_t it = 0, tc = 0;
      bool ok = true;
      auto commit = [&](uint32_t bar) {
        if constexpr (CTAS == 2) ptx::mma_commit_pair(bar, (uint16_t)3); else ptx::mma_commit(bar);
      };
      uint32_t un_seq = 0;
      int u = take_unit(0);
      for (; u >= 0 && ok; u = take_unit(++un_seq)) {
        const Unit un = decode_unit(p, m_tiles, u);
        for (int n = un.n_begin; n < un.n_end && ok; ++n) {
          const int acc = tc & 1;
          const uint32_t aph = (tc >> 1) & 1u;
          if (!ptx::mbar_wait(tempty_bar(acc), aph ^ 1u, abort, WAIT_LIMIT_NS)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * TN;
          for (int kb0 = 0; kb0 < k_blocks; kb0 += SUBS) {
            const int s = it % NSTAGE;
            const uint32_t ph = (it / NSTAGE) & 1u;
            if (!ptx::mbar_wait(full_bar(s), ph, abort, WAIT_LIMIT_NS)) { ok = false; break; }
            ptx::tc_fence_after();
#pragma unroll
            for (int sub = 0; sub < SUBS; ++sub) {
              const uint32_t sa = smem_base + s * STAGE + sub * SUB, sb = sa + A_BYTES;
#pragma unroll
              for (int k = 0; k < TK / 16; ++k) {
                // K-major: 16 elements = 32 B further along the swizzled 128 B row.
                // MN-major: 16 k-rows of 128 B = two 8-row swizzle atoms further.
                const uint64_t da = A_MN ? ptx::make_smem_desc(sa + k * 2048, SUB_BYTES, 1024)
                                         : ptx::make_smem_desc(sa + k * 32, 16, 1024);
                const uint64_t db = B_MN ? ptx::make_smem_desc(sb + k * 2048, SUB_BYTES, 1024)
                                         : ptx::make_smem_desc(sb + k * 32, 16, 1024);
                const uint32_t accum = (kb0 | sub | k) != 0 ? 1u : 0u;
                if constexpr (CTAS == 2) ptx::mma_bf16_ss_pair(d_tmem, da, db, IDESC, accum);
                else ptx::mma_bf16_ss(d_tmem, da, db, IDESC, accum);
              }
            }
            commit(empty_bar(s));  // frees the stage (in both CTAs) once these MMAs have read it
            ++it;
          }
          if (!ok) break;
          commit(tfull_bar(acc));  // accumulator complete (in both CTAs)
          ++tc;
        }
        if (!ok) break;
      }
      if (u == -2) ok = false;
      if (!ok) {
        if constexpr (CTAS == 2) ptx::mma_commit_pair(done_bar, (uint16_t)1); else ptx::mma_commit(done_bar);
        ptx::mbar_wait(done_bar, 0, nullptr, DRAIN_LIMIT_NS);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int q = warp & 3;  // tensor-memory lane quarter this warp may read
    uint32_t tc = 0;
    bool ok = true;
    // warp-collective form of take_unit
    auto take_unit_warp = [&](uint32_t n) -> int {
      if (!dynamic) return static_unit(n);
      const int slot = n % SCHED_SLOTS;
      if (!mbar_wait_warp<true>(ufull_bar(slot), (n / SCHED_SLOTS) & 1u, abort, lane)) return -2;
      const int u = unit_slot[slot];
      __syncwarp();
      if (lane == 0) {
        if (CTAS == 2 && !leader) ptx::mbar_arrive_remote(uempty_bar(slot), 0);
        else ptx::mbar_arrive(uempty_bar(slot));
      }
      return u;
    };
    // TMA-written outputs: this warp's two staging boxes, and how many boxes it has handed over so far
    const uint32_t out_stage = smem_base + RING_BYTES + (uint32_t)(warp - 2) * 2 * OUT_BOX_BYTES;
    const uint32_t out_row = out_stage + (uint32_t)lane * 128u;   // this lane's 128-byte row within box 0
    uint32_t boxes = 0;
    if constexpr (MODE != FWD) {
      if (p.out_tma && lane == 0) ptx::prefetch_tensormap(&tmC);
    }
    // Box protocol (all lanes call, lane 0 talks to the TMA unit).  begin: the box to fill next was the source
    // of the store issued two boxes ago, wait until that one has read it.  put: 16 bytes at chunk j of this
    // lane's row, at the position the 128-byte swizzle gives it.  end: publish the writes to the async proxy
    // and issue the store (or the add) of the box at tensor coordinates (x, y).
    auto box_begin = [&]() {
      if (lane == 0) ptx::bulk_wait_group_read<1>();
      __syncwarp();
    };
    auto box_put = [&](int j, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
      ptx::st_shared_v4(out_row + (boxes & 1u) * OUT_BOX_BYTES + (uint32_t)((j ^ (lane & 7)) << 4), a, b, c, d);
    };
    auto box_end = [&](int x, int y) {
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        const uint32_t src = out_stage + (boxes & 1u) * OUT_BOX_BYTES;
        // checked build: the box starts inside the output (what sticks out past its extents is clipped by the store)
        if (DRK_IN_RANGE(x >= 0 && x < p.cols && y >= 0 && y < rows, p.status)) {
          if (p.out_tma == 2) ptx::tma_reduce_add_2d(&tmC, src, x, y);
          else ptx::tma_store_2d(&tmC, src, x, y);
        }
        ptx::bulk_commit_group();
      }
      ++boxes;
    };
    uint32_t un_seq = 0;
    for (int u = take_unit_warp(0); u >= 0 && ok; u = take_unit_warp(++un_seq)) {
      const Unit un = decode_unit(p, m_tiles, u);
      const int64_t row = ((int64_t)un.m * CTAS + cta_rank) * TM + q * 32 + lane;
      const int slab_row0 = (un.m * CTAS + cta_rank) * TM + q * 32;   // first row of this warp's 32-row slab
      bool row_ok = row < rows;
      // orow: the token this accumulator row belongs to (differs from row when rows are compacted)
      int64_t orow = row;
      if constexpr (MODE == FWD || MODE == DL || MODE == DH) {
        if (p.rowmap != nullptr) orow = row_ok ? (int64_t)p.rowmap[row] : -1;
        if constexpr (MODE == DH || MODE == FWD) row_ok = row_ok && orow >= 0;
        // checked build: the token a compacted row maps to lies inside the batch, the unit inside the grid of units
        if (!DRK_IN_RANGE((p.rowmap == nullptr || orow < p.T) && un.m < m_tiles && un.j < p.nj, p.status)) {
          row_ok = false;
          orow = -1;
        }
      }
      // per-unit state
      float run_m = -CUDART_INF_F, run_l = 0.f, run_r = 0.f;  // FWD: log2-domain running max, sum, sum*logit
      int id = -1;
      float c_t = 0.f, z2 = 0.f;
      if constexpr (MODE == FWD) {
        if (row_ok) id = local_id(p.ids[orow], p.id_off, p.id_width);   // partials and target logits stay indexed by the (compact) row
      }
      if constexpr (MODE == DL) {
        if (row_ok && orow >= 0) { id = local_id(p.ids[orow], p.id_off, p.id_width); c_t = p.coeff[orow]; z2 = p.lse[orow] * kLog2e; }
      }
      for (int n = un.n_begin; n < un.n_end; ++n) {
        const int acc = tc & 1;
        const uint32_t aph = (tc >> 1) & 1u;
        if (!mbar_wait_warp(tfull_bar(acc), aph, abort, lane)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * TN;
#pragma unroll 1
        for (int c = 0; c < TN / 32; ++c) {
          uint32_t raw[32];
          __syncwarp();
          ptx::tmem_ld_32x32(taddr + c * 32, raw);
          ptx::tmem_ld_wait();
          float x[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) x[j] = __uint_as_float(raw[j]);
          const int col = n * TN + c * 32;  // column index within [0, cols)
          if constexpr (MODE == FWD) {
            if (col + 32 > p.cols) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col + j >= p.cols) x[j] = -CUDART_INF_F;
            }
            if ((uint32_t)(id - col) < 32u) {
              const int w = id - col;
              float tg = 0.f;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j == w) tg = x[j];
              if (DRK_IN_RANGE(row < p.T, p.status)) p.tgt[row] = tg;
            }
            float cm = x[0];
#pragma unroll
            for (int j = 1; j < 32; ++j) cm = fmaxf(cm, x[j]);
            const float m_new = fmaxf(run_m, cm * kLog2e);
            if (m_new > -CUDART_INF_F) {
              float s = 0.f;
              const float resc = ex2(run_m - m_new);
              if (p.want_entropy) {
                float sx = 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  const float e = ex2(fmaf(x[j], kLog2e, -m_new));
                  s += e;
                  sx = fmaf(e, fmaxf(x[j], -3.0e38f), sx);   // masked columns (-inf) contribute 0
                }
                run_r = run_r * resc + sx;
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) s += ex2(fmaf(x[j], kLog2e, -m_new));
              }
              run_l = run_l * resc + s;
              run_m = m_new;
            }
          } else if constexpr (MODE == DL) {
            // dL = c_t (softmax - onehot) for 32 columns of this lane's row
            auto dl_values = [&]() {
              const int gcol = p.v0 + col;
              if (row_ok && c_t != 0.f) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  const float pr = ex2(fmaf(x[j], kLog2e, -z2));
                  x[j] = c_t * (pr - ((gcol + j == id) ? 1.f : 0.f));
                }
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) x[j] = 0.f;
              }
            };
            if (p.out_tma) {
              // two 32-column blocks make one box of 64 bf16 columns (128 bytes per row); columns past the
              // chunk's width are clipped by the store
              const int pair_col = n * TN + (c & ~1) * 32;
              if (slab_row0 < rows && pair_col < p.cols) {
                dl_values();
                if ((c & 1) == 0) box_begin();
#pragma unroll
                for (int qd = 0; qd < 4; ++qd)
                  box_put((c & 1) * 4 + qd, pack_bf16(x[qd * 8 + 0], x[qd * 8 + 1]), pack_bf16(x[qd * 8 + 2], x[qd * 8 + 3]),
                          pack_bf16(x[qd * 8 + 4], x[qd * 8 + 5]), pack_bf16(x[qd * 8 + 6], x[qd * 8 + 7]));
                if (c & 1) box_end(pair_col, slab_row0);
              }
            } else if (row_ok && col < p.cols) {
              dl_values();
              __nv_bfloat16* dst = p.dL + row * p.vc + col;
              if (col + 32 <= p.cols) {
                uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
                for (int qd = 0; qd < 4; ++qd)
                  d4[qd] = make_uint4(pack_bf16(x[qd * 8 + 0], x[qd * 8 + 1]), pack_bf16(x[qd * 8 + 2], x[qd * 8 + 3]),
                                      pack_bf16(x[qd * 8 + 4], x[qd * 8 + 5]), pack_bf16(x[qd * 8 + 6], x[qd * 8 + 7]));
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (col + j < p.cols) dst[j] = __float2bfloat16(x[j]);
              }
            }
          } else {  // DW, DH
            if constexpr (MODE == DW) {
              if (k_blocks == 0) {  // nothing to contract over: the accumulator was never written
#pragma unroll
                for (int j = 0; j < 32; ++j) x[j] = 0.f;
              }
            }
            if (p.out_tma) {
              // rows past the output's extent (ragged vocabulary tail) and columns past H are clipped by the store
              if (p.out_bf16) {
                const int pair_col = n * TN + (c & ~1) * 32;
                if (slab_row0 < rows && pair_col < p.cols) {
                  if ((c & 1) == 0) box_begin();
#pragma unroll
                  for (int qd = 0; qd < 4; ++qd)
                    box_put((c & 1) * 4 + qd, pack_bf16(x[qd * 8 + 0], x[qd * 8 + 1]), pack_bf16(x[qd * 8 + 2], x[qd * 8 + 3]),
                            pack_bf16(x[qd * 8 + 4], x[qd * 8 + 5]), pack_bf16(x[qd * 8 + 6], x[qd * 8 + 7]));
                  if (c & 1) box_end(pair_col, slab_row0);
                }
              } else if (slab_row0 < rows && col < p.cols) {
                box_begin();
#pragma unroll
                for (int qd = 0; qd < 8; ++qd)
                  box_put(qd, raw_bits(x[qd * 4 + 0]), raw_bits(x[qd * 4 + 1]), raw_bits(x[qd * 4 + 2]), raw_bits(x[qd * 4 + 3]));
                box_end(col, slab_row0);
              }
            } else if (row_ok && col < p.cols) {
              store_row_chunk(p, orow, col, x);
            }
          }
        }
        // this warp has drained its quarter of the accumulator: tell the MMA issuer (even CTA)
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (CTAS == 2 && !leader) ptx::mbar_arrive_remote(tempty_bar(acc), 0);
          else ptx::mbar_arrive(tempty_bar(acc));
        }
        ++tc;
      }
      if (!ok) break;
      if constexpr (MODE == FWD) {
        if (row_ok) {
          // natural-log units for the max, as the merge kernel expects
          if (DRK_IN_RANGE(row < p.T && un.j < p.nj, p.status))
            reinterpret_cast<float4*>(p.part)[(int64_t)un.j * p.T + row] = make_float4(run_m * kLn2, run_l, run_r, 0.f);
        }
      }
    }
    // every store this warp issued has been performed before the block (and its shared memory) goes away
    if constexpr (MODE != FWD) {
      if (lane == 0) ptx::bulk_wait_group<0>();
      __syncwarp();
    }
  }

  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before();
  // In a pair neither CTA may leave (or free tensor memory) while its peer can still address it.
  if constexpr (CTAS == 2) ptx::cluster_sync(); else __syncthreads();
  if (threadIdx.x == 0 && *abort) atomicOr(p.status, DRK_STATUS_TIMEOUT);
  if (warp == 1) {
    ptx::tc_fence_after();
    if constexpr (CTAS == 2) ptx::tmem_dealloc_pair(tmem_base, 512); else ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Self-test of the bounded waits: one block waits on an mbarrier on which nothing ever arrives.  Lane 0 of
// warp 0 waits like the producer and MMA threads do and gives up after limit_ns, raising the block's abort
// flag; warp 1 waits like an epilogue warp (its own limit is WAIT_LIMIT_NS) and must leave as soon as it
// sees the flag.  The block then reports DRK_STATUS_TIMEOUT exactly as the GEMM kernels do.
__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint64_t limit_ns, uint64_t* waited_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  const uint32_t bar_addr = ptx::smem_u32(&bar);
  volatile int* abort = &abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_addr, 1);
    *abort = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t t0 = ptx::globaltimer_ns();
  bool ok = true;
  if (warp == 0) {
    if (lane == 0) ok = ptx::mbar_wait(bar_addr, 0, abort, limit_ns);
  } else {
    ok = mbar_wait_warp(bar_addr, 0, abort, lane);
  }
  const uint64_t waited = ptx::globaltimer_ns() - t0;
  if (lane == 0) waited_ns[warp] = waited;
  __syncthreads();
  if (threadIdx.x == 0 && (*abort || !ok)) atomicOr(status, DRK_STATUS_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

// Tensor maps depend on the address and geometry only, never on the contents, so a map encoded once serves
// every later call on the same buffer: a steady-state training step (same W, hidden and workspace pointers)
// encodes nothing.  One table for the process, shared by all threads; emptied when it reaches kMapLimit
// entries (a caller cycling through thousands of distinct buffers simply re-encodes).
struct MapKey {
  const void* base; uint64_t inner, outer, pitch_bytes; uint32_t box_inner, box_outer, dtype;
  bool operator==(const MapKey& o) const {
    return base == o.base && inner == o.inner && outer == o.outer && pitch_bytes == o.pitch_bytes &&
           box_inner == o.box_inner && box_outer == o.box_outer && dtype == o.dtype;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    uint64_t h = reinterpret_cast<uintptr_t>(k.base) * 0x9E3779B97F4A7C15ull;
    h ^= (k.inner + 0x632BE59BD9B4E019ull) * 0xFF51AFD7ED558CCDull;
    h ^= (k.outer + (h >> 29)) * 0xC4CEB9FE1A85EC53ull;
    h ^= ((uint64_t)k.box_inner << 40) ^ ((uint64_t)k.box_outer << 20) ^ k.dtype ^ (k.pitch_bytes * 0x2545F4914F6CDD1Dull);
    return (size_t)(h ^ (h >> 32));
  }
};
constexpr size_t kMapLimit = 8192;
std::mutex g_map_mu;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash>& map_table() {
  static auto* t = new std::unordered_map<MapKey, CUtensorMap, MapKeyHash>();   // never destroyed: no exit-order issues
  return *t;
}
std::atomic<uint64_t> g_map_encodes{0};
// Host-side fault injection for tests: when positive, the n-th next request for a tensor map fails as if the
// driver had refused to encode it (cached or not).
std::atomic<int> g_fail_map_in{0};

// Row-major matrix [outer, inner] of 2-byte (bf16) or 4-byte (fp32) elements with row pitch `pitch_elems`;
// box = box_inner x box_outer, 128-byte swizzle, zero fill outside the extents on loads (stores are clipped).
bool make_map_typed(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer, uint64_t pitch_elems,
                    uint32_t box_inner, uint32_t box_outer, bool f32) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if (g_fail_map_in.load(std::memory_order_relaxed) > 0 && g_fail_map_in.fetch_sub(1) == 1) return false;
  const uint32_t esz = f32 ? 4 : 2;
  const MapKey key{base, inner, outer, pitch_elems * esz, box_inner, box_outer, f32 ? 1u : 0u};
  {
    std::lock_guard<std::mutex> lock(g_map_mu);
    auto& t = map_table();
    auto it = t.find(key);
    if (it != t.end()) { *m = it->second; return true; }
  }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {pitch_elems * esz};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  if (fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
         strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  g_map_encodes.fetch_add(1, std::memory_order_relaxed);
  std::lock_guard<std::mutex> lock(g_map_mu);
  auto& t = map_table();
  if (t.size() >= kMapLimit) t.clear();
  t.emplace(key, *m);
  return true;
}

bool make_map(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer, uint64_t pitch_elems,
              uint32_t box_inner, uint32_t box_outer) {
  return make_map_typed(m, base, inner, outer, pitch_elems, box_inner, box_outer, false);
}

template <int MODE, int CTAS>
__global__ void umma_gemm_kernel(const __grid_constant__ CUtensorMap, const __grid_constant__ CUtensorMap,
                                 const __grid_constant__ CUtensorMap, const UmmaParams);

// How many two-CTA clusters of this kernel the device can hold at once (one CTA per SM); 0 if the query fails.
int resident_pairs() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return sm_count() / 2;
  if (cached[dev] > 0) return cached[dev];
  auto kern = umma_gemm_kernel<0, 2>;
  int n = 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(sm_count() / 2 * 2);
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    n = sm_count() / 2;
  }
  if (n > sm_count() / 2) n = sm_count() / 2;
  cached[dev] = n;
  return n;
}

template <int MODE, int CTAS>
bool set_smem_attr() {
  if (cudaFuncSetAttribute(umma_gemm_kernel<MODE, CTAS>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) !=
      cudaSuccess) {
    (void)cudaGetLastError();
    return false;
  }
  return true;
}

// Everything on the host that can fail and does not depend on the call's arguments: the driver entry point
// for tensor-map encoding, the shared-memory attribute of all eight kernel instantiations, and the
// residency query.  Done once per device; later calls return the cached answer.
int umma_prepare() {
  static std::mutex mu;
  static int state[64] = {};   // 0 unknown, 1 ready, -1 failed
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DRK_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (state[dev] == 0) {
    bool ok = get_encode_fn() != nullptr;
    ok = ok && set_smem_attr<FWD, 1>() && set_smem_attr<DL, 1>() && set_smem_attr<DW, 1>() && set_smem_attr<DH, 1>();
    ok = ok && set_smem_attr<FWD, 2>() && set_smem_attr<DL, 2>() && set_smem_attr<DW, 2>() && set_smem_attr<DH, 2>();
    if (ok) (void)resident_pairs();
    state[dev] = ok ? 1 : -1;
  }
  return state[dev] == 1 ? DRK_OK : DRK_ERR_CUDA;
}

// a, b: operand maps; c: the output map of the TMA-written epilogues (any valid map where out_tma is 0).
template <int MODE, int CTAS>
int launch_mode_ctas(const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c, UmmaParams p, cudaStream_t st) {
  p.num_units = p.m_tiles * p.nj;   // upper bound when the row count lives on the device
  if (p.num_units <= 0) return DRK_OK;
  auto kern = umma_gemm_kernel<MODE, CTAS>;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (CTAS == 2) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int pairs = resident_pairs();
    cfg.gridDim = dim3(2 * (p.num_units < pairs ? p.num_units : pairs));
  } else {
    cfg.gridDim = dim3(p.num_units < sm_count() ? p.num_units : sm_count());
  }
  if (cudaLaunchKernelEx(&cfg, kern, a, b, c, p) != cudaSuccess) { (void)cudaGetLastError(); return DRK_ERR_CUDA; }
  DRK_LAUNCHED();
  return DRK_OK;
}

template <int MODE>
int launch_mode(int ctas, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c, const UmmaParams& p,
                cudaStream_t st) {
  return ctas == 2 ? launch_mode_ctas<MODE, 2>(a, b, c, p, st) : launch_mode_ctas<MODE, 1>(a, b, c, p, st);
}

}  // namespace

uint64_t umma_map_encodes() { return g_map_encodes.load(std::memory_order_relaxed); }
void umma_fail_map_request(int nth) { g_fail_map_in.store(nth > 0 ? nth : 0); }

// Number of vocabulary ranges per row tile in the forward (each work unit = one row tile x one range,
// with its own partial max / sum-exp per row).
//  - default: ranges of two 256-column tiles.  Short units, taken in an order that keeps ~38 MB of hidden
//    panels (a group of row tiles) live while the group sweeps the vocabulary, let L2 serve most operand
//    re-reads: measured at T=32768, H=5120, V=151936 the forward dropped from ~44 to ~38.5 ms against four
//    long ranges per row tile, and to 35.5 ms (16 GB of DRAM reads) once the units were drawn dynamically.
//  - frugal: the fewest ranges that fill whole waves (within 1 % of the best wave efficiency), for
//    callers with little scratch for the partials.
int umma_nsplit(int64_t T, int V, int ctas, bool frugal) {
  const int64_t m_tiles = ceil_div(T, TM * ctas);
  const int n_tiles = (int)ceil_div(V, TN);
  if (m_tiles <= 0) return 1;
  if (!frugal) {
    // ranges of two tiles, longer ones where the partials (16 bytes per row and range) would pass 256 MiB
    int64_t cap = ((int64_t)1 << 28) / (16 * T);
    if (cap < 32) cap = 32;
    int64_t per = 2;
    if (ceil_div(n_tiles, per) > cap) per = ceil_div(n_tiles, cap);
    return (int)ceil_div(n_tiles, per);
  }
  const int sms = sm_count() / ctas;
  double eff[33];
  double best_eff = -1.0;
  for (int ns = 1; ns <= 32; ++ns) {
    eff[ns] = -1.0;
    if (ns > n_tiles) continue;
    const int per = (int)ceil_div(n_tiles, ns);
    if ((int)ceil_div(n_tiles, per) != ns) continue;
    if (per < 4 && ns > 1) continue;
    const int64_t waves = ceil_div(m_tiles * ns, sms);
    // time ~ waves * per tiles; work = m_tiles * n_tiles tiles
    eff[ns] = (double)(m_tiles * (int64_t)n_tiles) / ((double)waves * per * sms);
    if (eff[ns] > best_eff) best_eff = eff[ns];
  }
  for (int ns = 1; ns <= 32; ++ns)
    if (eff[ns] >= best_eff - 0.01) return ns;
  return 1;
}

// How many operand panels (rows x K bf16 each) a group of work units keeps live in L2 while the other
// operand streams past: about 38 MB worth.  Measured at T=32768, H=5120, V=151936 (interleaved runs): 10 column
// tiles for DH (7424-deep panels) and 12-15 for DL are 2.7 % faster than row-tile groups that sweep all columns;
// 20 and more fall off again, as do forward groups beyond ~16 row tiles (L2 serves both dies from 126 MB).
static int panel_group(int rows_per_tile, int64_t k_elems) {
  const double panel = (double)rows_per_tile * (double)k_elems * 2.0;
  int g = (int)(38.0 * 1024 * 1024 / panel);
  return g < 1 ? 1 : (g > 64 ? 64 : g);
}

int launch_bounded_wait_selftest(uint32_t limit_ms, uint32_t* status, uint64_t* waited_ns, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(status, (uint64_t)limit_ms * 1000000ull, waited_ns);
  DRK_LAUNCHED();
  return DRK_OK;
}

// ---- forward ----------------------------------------------------------------------------------------------

int plan_umma_fwd(const UmmaFwdArgs& a, UmmaFwdPlan* plan) {
  int rc = umma_prepare();
  if (rc != DRK_OK) return rc;
  plan->a = a;
  const int ctas = a.ctas == 2 ? 2 : 1;
  // With a row map the forward runs over the gathered rows (hidden_c) only; the kernels read their number.
  const void* hid = a.rowmap ? (const void*)a.hidden_c : a.hidden;
  const int64_t hid_rows = a.rowmap ? ceil_div(a.T, 256) * 256 : a.T;
  if (!make_map(&plan->mh, hid, a.H, hid_rows, a.H, TK, TM)) return DRK_ERR_CUDA;
  if (!make_map(&plan->mw, a.W, a.H, a.V, a.H, TK, TN / ctas)) return DRK_ERR_CUDA;
  return DRK_OK;
}

int enqueue_umma_fwd(const UmmaFwdPlan& plan, cudaStream_t st) {
  const UmmaFwdArgs& a = plan.a;
  const int ctas = a.ctas == 2 ? 2 : 1;
  UmmaParams p{};
  p.m_tiles = (int)ceil_div(a.T, TM * ctas);
  p.n_tiles = (int)ceil_div(a.V, TN);
  p.k_blocks = (int)ceil_div(a.H, TK);
  p.nj = a.nsplit;
  p.tiles_per_unit = (int)ceil_div(p.n_tiles, a.nsplit);
  const int slots = sm_count() / ctas;
  if (a.nsplit > 32 || a.nsplit * 8 >= p.n_tiles) p.group_m = panel_group(TM * ctas, a.H);  // short units: panel budget
  else p.group_m = slots / a.nsplit > 0 ? slots / a.nsplit : 1;                    // long ranges: one wave
  p.rows = a.T; p.cols = a.V; p.v0 = 0; p.T = a.T;
  p.id_off = a.id_off; p.id_width = a.V;
  p.ids = a.ids; p.part = a.part; p.tgt = a.tgt; p.status = a.status;
  p.want_entropy = a.entropy != nullptr || a.stats != nullptr;   // the statistics carry the same third sum
  p.rowmap = a.rowmap; p.n_rows = a.n_rows;
  p.sched = a.sched;
  if (a.sched != nullptr) DRK_CUDA_CHECK(cudaMemsetAsync(a.sched, 0, sizeof(int32_t), st));
  int rc = launch_mode<FWD>(ctas, plan.mh, plan.mw, plan.mh, p, st);
  if (rc != DRK_OK) return rc;
  if (a.stats != nullptr)
    return launch_shard_stats(a.part, a.tgt, a.ids, a.id_off, a.T, a.V, a.nsplit, a.stats, a.status, st);
  return launch_lse_merge(a.part, a.tgt, a.ids, a.T, a.V, a.nsplit, a.logp, a.lse, a.entropy, a.status, a.rowmap,
                          a.n_rows, st);
}

int launch_umma_fwd(const UmmaFwdArgs& a, cudaStream_t st) {
  UmmaFwdPlan plan;
  int rc = plan_umma_fwd(a, &plan);
  if (rc != DRK_OK) return rc;
  return enqueue_umma_fwd(plan, st);
}

// ---- backward ---------------------------------------------------------------------------------------------

int plan_umma_bwd(const UmmaBwdArgs& a, UmmaBwdPlan* plan) {
  int rc = umma_prepare();
  if (rc != DRK_OK) return rc;
  plan->a = a;
  const int ctas = a.ctas == 2 ? 2 : 1;
  // The row dimension of the three contractions runs over the compacted rows (hidden_c, rowmap);
  // buffers are sized for the worst case (every row kept), the kernels read the actual count.
  const int64_t rows_cap = ceil_div(a.T, 256) * 256;
  if (!make_map(&plan->mh_k, a.hidden_c, a.H, rows_cap, a.H, TK, TM)) return DRK_ERR_CUDA;
  if (!make_map(&plan->mw_k, a.W, a.H, a.V, a.H, TK, TN / ctas)) return DRK_ERR_CUDA;
  if (!make_map(&plan->mh_mn, a.hidden_c, a.H, rows_cap, a.H, 64, TK)) return DRK_ERR_CUDA;
  if (!make_map(&plan->mw_mn, a.W, a.H, a.V, a.H, 64, TK)) return DRK_ERR_CUDA;
  const int n_chunks = (int)ceil_div(a.V, a.vc);
  plan->mdl_k.resize(n_chunks);
  plan->mdl_mn.resize(n_chunks);
  plan->mdl_out.resize(n_chunks);
  plan->mdw_out.resize(n_chunks);
  // Output boxes of the epilogues: 32 rows x 128 bytes (64 bf16 or 32 fp32 columns).
  const bool dw_f32 = a.dw_dtype == DRK_F32;
  plan->dw_out_tma = !a.dw_accumulate ? 1 : (dw_f32 ? 2 : 0);   // bf16 accumulation keeps the register path
  for (int c = 0; c < n_chunks; ++c) {
    const int v0 = c * a.vc;
    const int vc_this = a.V - v0 < a.vc ? a.V - v0 : a.vc;
    if (!make_map(&plan->mdl_k[c], a.dL, vc_this, rows_cap, a.vc, TK, TM)) return DRK_ERR_CUDA;
    if (!make_map(&plan->mdl_mn[c], a.dL, vc_this, rows_cap, a.vc, 64, TK)) return DRK_ERR_CUDA;
    if (!make_map(&plan->mdl_out[c], a.dL, vc_this, rows_cap, a.vc, 64, 32)) return DRK_ERR_CUDA;
    const void* dw_rows = (const char*)a.dW + (size_t)v0 * a.H * (dw_f32 ? 4 : 2);
    if (!make_map_typed(&plan->mdw_out[c], dw_rows, a.H, vc_this, a.H, dw_f32 ? 32 : 64, 32, dw_f32)) return DRK_ERR_CUDA;
  }
  // dH is accumulated in fp32 over the compacted rows and scattered to the tokens' rows at the end
  if (!make_map_typed(&plan->mdh_out, a.dH_acc, a.H, rows_cap, a.H, 32, 32, true)) return DRK_ERR_CUDA;
  return DRK_OK;
}

int enqueue_umma_bwd(const UmmaBwdPlan& plan, cudaStream_t st) {
  const UmmaBwdArgs& a = plan.a;
  const int ctas = a.ctas == 2 ? 2 : 1;
  const int TMC = TM * ctas;   // rows of one work unit's tile
  // rows that are not in the compacted set keep this zero
  DRK_CUDA_CHECK(cudaMemsetAsync(a.dH, 0, (size_t)a.T * a.H * (a.dh_dtype == DRK_BF16 ? 2 : 4), st));
  const int n_chunks = (int)ceil_div(a.V, a.vc);
  // one work counter per launch (three per vocabulary chunk), all cleared by one memset
  if (a.sched != nullptr) DRK_CUDA_CHECK(cudaMemsetAsync(a.sched, 0, sizeof(int32_t) * 3 * (size_t)n_chunks, st));
  int chunk = 0;
  for (int v0 = 0; v0 < a.V; v0 += a.vc, ++chunk) {
    const int vc_this = a.V - v0 < a.vc ? a.V - v0 : a.vc;
    const CUtensorMap& mdl_k = plan.mdl_k[chunk];
    const CUtensorMap& mdl_mn = plan.mdl_mn[chunk];
    {  // dL chunk = c (softmax - onehot), recomputed from hidden W^T
      UmmaParams p{};
      p.m_tiles = (int)ceil_div(a.T, TMC);
      p.n_tiles = (int)ceil_div(vc_this, TN);
      p.k_blocks = (int)ceil_div(a.H, TK);
      p.nj = p.n_tiles; p.tiles_per_unit = 1; p.group_m = 16 / ctas;
      p.group_n = panel_group(TN, a.H);        // W's column panels of the group stay in L2, the rows stream past
      p.rows = a.T; p.cols = vc_this; p.v0 = v0; p.T = a.T;
      p.id_off = a.id_off; p.id_width = a.V;
      p.ids = a.ids; p.lse = a.lse; p.coeff = a.coeff; p.dL = a.dL; p.vc = a.vc; p.status = a.status;
      p.rowmap = a.rowmap; p.n_rows = a.n_rows;
      p.out_tma = 1; p.out_bf16 = 1;
      p.sched = a.sched ? a.sched + 3 * chunk : nullptr;
      int rc = launch_mode<DL>(ctas, plan.mh_k, plan.mw_k, plan.mdl_out[chunk], p, st);
      if (rc != DRK_OK) return rc;
    }
    {  // dW[v0 : v0 + vc_this, :] (+)= dL^T hidden
      UmmaParams p{};
      p.m_tiles = (int)ceil_div(vc_this, TMC);
      p.n_tiles = (int)ceil_div(a.H, TN);
      p.k_blocks = (int)ceil_div(a.T, TK);
      p.nj = p.n_tiles; p.tiles_per_unit = 1; p.group_m = 16 / ctas;
      p.rows = vc_this; p.cols = a.H; p.v0 = v0; p.T = a.T;
      const size_t esz = a.dw_dtype == DRK_BF16 ? 2 : 4;
      p.C = (char*)a.dW + (size_t)v0 * a.H * esz; p.C_in = p.C; p.ldc = a.H;
      p.beta = a.dw_accumulate; p.out_bf16 = a.dw_dtype == DRK_BF16; p.in_bf16 = p.out_bf16;
      p.out_tma = plan.dw_out_tma;
      p.status = a.status;
      p.rowmap = a.rowmap; p.n_rows = a.n_rows;
      p.sched = a.sched ? a.sched + 3 * chunk + 1 : nullptr;
      int rc = launch_mode<DW>(ctas, mdl_mn, plan.mh_mn, plan.mdw_out[chunk], p, st);
      if (rc != DRK_OK) return rc;
      if (a.chunk_events != nullptr)
        DRK_CUDA_CHECK(cudaEventRecord(static_cast<cudaEvent_t>(a.chunk_events[chunk]), st));
    }
    {  // dH_acc (+)= dL W[v0 : v0 + vc_this, :], over the compacted rows: stored by the first chunk, added to by the rest
      UmmaParams p{};
      p.m_tiles = (int)ceil_div(a.T, TMC);
      p.n_tiles = (int)ceil_div(a.H, TN);
      p.k_blocks = (int)ceil_div(vc_this, TK);
      p.nj = p.n_tiles; p.tiles_per_unit = 1; p.group_m = 32 / ctas;
      // the W chunk's column panels of the group stay in L2 where they fit; with deep chunks (long panels) at
      // least ten column tiles per group keep the set of tiles in flight about square (rows x columns)
      p.group_n = panel_group(TN, vc_this);
      if (p.group_n < 10) p.group_n = 10;
      p.rows = a.T; p.cols = a.H; p.v0 = v0; p.T = a.T;
      p.ldc = a.H; p.out_bf16 = 0; p.out_tma = chunk > 0 ? 2 : 1;
      p.status = a.status;
      p.rowmap = nullptr; p.n_rows = a.n_rows;
      p.sched = a.sched ? a.sched + 3 * chunk + 2 : nullptr;
      int rc = launch_mode<DH>(ctas, mdl_k, plan.mw_mn, plan.mdh_out, p, st);
      if (rc != DRK_OK) return rc;
    }
  }
  // dH[rowmap[r], :] = dH_acc[r, :] in the requested type
  return launch_scatter_rows(a.dH_acc, a.H, a.rowmap, a.n_rows, a.dH, a.dh_dtype == DRK_BF16, a.T, a.status, st);
}

int launch_umma_bwd(const UmmaBwdArgs& a, cudaStream_t st) {
  UmmaBwdPlan plan;
  int rc = plan_umma_bwd(a, &plan);
  if (rc != DRK_OK) return rc;
  return enqueue_umma_bwd(plan, st);
}

}  // namespace drk
