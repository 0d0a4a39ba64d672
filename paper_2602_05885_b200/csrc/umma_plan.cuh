// Host-side plans of the tcgen05 path: everything a call needs that can fail on the host (driver entry point,
// kernel attributes, tensor-map encoding) is done while the plan is built, before anything is enqueued.
#pragma once
#include "common.cuh"
#include <cuda.h>
#include <vector>

namespace drk {

struct UmmaFwdPlan {
  UmmaFwdArgs a;
  CUtensorMap mh, mw;   // hidden (or the gathered rows) and W, K-major boxes
};
int plan_umma_fwd(const UmmaFwdArgs& a, UmmaFwdPlan* plan);       // enqueues nothing
int enqueue_umma_fwd(const UmmaFwdPlan& plan, cudaStream_t st);

struct UmmaBwdPlan {
  UmmaBwdArgs a;
  CUtensorMap mh_k, mw_k, mh_mn, mw_mn;       // gathered hidden rows and W, as K-major and as MN-major operands
  std::vector<CUtensorMap> mdl_k, mdl_mn;     // the dL buffer per vocabulary chunk (the last chunk is narrower)
  // outputs written by the TMA unit in boxes of 32 rows x 128 bytes: the dL chunk, the chunk's rows of dW, and
  // the fp32 accumulator of dH over the compacted rows
  std::vector<CUtensorMap> mdl_out, mdw_out;
  CUtensorMap mdh_out;
  int dw_out_tma;                             // 1 store, 2 add (fp32 accumulation), 0 register path
};
int plan_umma_bwd(const UmmaBwdArgs& a, UmmaBwdPlan* plan);       // enqueues nothing
int enqueue_umma_bwd(const UmmaBwdPlan& plan, cudaStream_t st);

// Tensor maps encoded so far by this process (cache misses); steady-state calls add none.
uint64_t umma_map_encodes();
// Test hook: the nth next tensor-map request fails (0 clears a pending injection).
void umma_fail_map_request(int nth);

}  // namespace drk
