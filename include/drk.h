/*
 * drk — fused policy-gradient loss over the LM head for multi-turn RL
 * (turn-level leave-one-out advantages + geometric mismatch rejection sampling).
 *
 * C ABI of libdrk.so.  Hand-written CUDA for sm_100a; one GPU per process.
 *
 * Conventions that hold for every entry point unless stated otherwise:
 *   - "device" pointers are CUDA device pointers of the current device; "host"
 *     pointers are ordinary host memory.  The caller owns every buffer, the
 *     workspace included; the library allocates nothing and keeps no state
 *     between calls apart from read-only per-process set-up (driver entry
 *     points, kernel attributes).
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream) and return without synchronising.  Scalar
 *     results (loss, counters, status) stay in device memory.
 *   - Return value: DRK_OK or a negative drk_status.  Arguments, sizes, the
 *     device's architecture, kernel attributes and every tensor map are checked
 *     or built on the host before the first enqueue: on DRK_ERR_INVALID_ARG,
 *     _UNSUPPORTED, _WORKSPACE or _ARCH nothing was enqueued, and DRK_ERR_CUDA
 *     from those host steps enqueues nothing either.  The one exception is
 *     DRK_ERR_CUDA raised by an enqueue itself (the runtime refusing a launch,
 *     a memset or an event record part-way through a call): earlier kernels of
 *     that call are then already on the stream and the outputs are undefined.
 *     Conditions only the device can see set bits in the device word `*status`
 *     (DRK_STATUS_*); no kernel traps or spins unbounded.
 *   - Sizes that depend on the device (workspace bytes, chunk widths) are
 *     computed for the current device's multiprocessor count.
 *   - All matrices are row-major and dense (leading dimension = row length).
 *   - Row t of `hidden` predicts the token `ids[t]`; the caller has already
 *     applied the next-token shift.
 */
#ifndef DRK_H_
#define DRK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DRK_OK = 0,
  DRK_ERR_INVALID_ARG = -1, /* null pointer, negative size, bad enum, misaligned pointer */
  DRK_ERR_UNSUPPORTED = -2, /* shape outside what the kernels handle (see each call)     */
  DRK_ERR_WORKSPACE = -3,   /* workspace_bytes smaller than drk_pg_workspace_bytes()     */
  DRK_ERR_CUDA = -4,        /* a CUDA runtime or driver call failed                       */
  DRK_ERR_ARCH = -5         /* current device is not compute capability 10.x             */
} drk_status;

typedef enum { DRK_F32 = 0, DRK_BF16 = 1 } drk_dtype;
typedef enum { DRK_BASELINE_TRLOO = 0, DRK_BASELINE_GRPO = 1 } drk_baseline;
typedef enum {
  DRK_NORM_KEPT_TOKENS = 0,       /* scale = 1 / (loss-masked tokens of retained samples), >= 1 */
  DRK_NORM_ALL_MASKED_TOKENS = 1, /* scale = 1 / (all loss-masked tokens inside segments), >= 1 */
  DRK_NORM_EXPLICIT = 2           /* scale = explicit_scale                                      */
} drk_norm;
typedef enum {
  DRK_ENGINE_AUTO = 0,     /* bf16 inputs: tcgen05 tensor-core kernels on CTA pairs (256x256 tiles);
                              fp32 inputs: fp32 FFMA kernels                                        */
  DRK_ENGINE_SIMT = 1,     /* force the FFMA kernels (exact fp32 products; slow; for cross-checks)  */
  DRK_ENGINE_UMMA_1CTA = 2 /* bf16 inputs: tcgen05 kernels with one CTA per 128x256 tile           */
} drk_engine;

typedef enum {
  DRK_SCHEDULE_DYNAMIC = 0, /* blocks draw their next work unit from a device-side counter as they finish one:
                               the units in flight are always consecutive, so the blocks that share an operand
                               panel through L2 stay together however unevenly they progress                */
  DRK_SCHEDULE_STATIC = 1   /* unit u belongs to block u mod (number of blocks), fixed at launch           */
} drk_schedule;

/* Bits of the device status word. */
#define DRK_STATUS_BAD_ID 1u       /* some ids[t] outside [0,V): that row's target logit reads as 0 */
#define DRK_STATUS_BAD_SEGMENTS 2u /* cu_seqlens not non-decreasing within [0,T]: segment skipped   */
#define DRK_STATUS_NONFINITE 4u    /* a non-finite log-sum-exp was produced                         */
#define DRK_STATUS_TIMEOUT 8u      /* a bounded on-chip wait expired; results are invalid           */
#define DRK_STATUS_BOUNDS 32u      /* checked build only (library compiled with -DDRK_BOUNDS_CHECK): an index
                                      derived on the device fell outside its array; the access was skipped    */
#define DRK_STATUS_BAD_GROUPS 16u  /* prompt_of_rollout decreases somewhere: a prompt's rollouts are not
                                      contiguous, so its turn groups were split (Sec. 4.2 groups by prompt) */

/*
 * Reward-to-go returns and turn-level advantages for a whole rollout batch
 * (Sec. 4.2: Eq. 2 for the return, Eq. 5 for TRLOO, Eq. 3 for the GRPO mean
 * baseline).
 *
 *   G[i,t]   = sum over valid t' >= t of gamma^(t'-t) * reward[i,t']
 *   group    = rollouts j with prompt_of_rollout[j] == prompt_of_rollout[i] and valid[j,t]
 *   TRLOO    : adv[i,t] = G[i,t] - mean_{j in group, j != i} G[j,t]   (0 when the group has one member)
 *   GRPO     : adv[i,t] = G[i,t] - mean_{j in group} G[j,t]
 *
 * reward, valid, ret, adv, gsize are [R*Tmax] device arrays indexed i*Tmax+t;
 * prompt_of_rollout is [R] device, non-decreasing (rollouts of a prompt are
 * contiguous): groups are the runs of equal values.  Where the array decreases,
 * a prompt whose rollouts are scattered would silently fall into several groups,
 * so that condition sets DRK_STATUS_BAD_GROUPS in *status (device uint32, OR-ed
 * into; may be NULL to skip the check).  Invalid (i,t) get ret = adv = 0 and
 * gsize = 0; valid ones get gsize = group size.  Arithmetic is fp64 inside,
 * outputs are rounded to fp32.  An all-equal group yields exactly 0.
 * R, Tmax >= 0 (0 enqueues nothing); Tmax <= 64, else DRK_ERR_UNSUPPORTED.
 * gamma must lie in [0,1].
 */
int drk_trloo_advantage(const float* reward, const uint8_t* valid,
                        const int32_t* prompt_of_rollout, int32_t R, int32_t Tmax,
                        float gamma, int32_t baseline, float* ret, float* adv,
                        int32_t* gsize, uint32_t* status, void* stream);

/*
 * Per-sample advantages of a packed micro-batch.  Every turn of a trajectory is one training sample
 * (Sec. 4.3); segment g holds turn seg_turn[g] of rollout seg_rollout[g] and takes
 *   seg_adv[g] = adv[seg_rollout[g] * Tmax + seg_turn[g]]
 * from the table drk_trloo_advantage wrote.  adv [R*Tmax] float, seg_rollout, seg_turn [S] int32, seg_adv [S]
 * float, status [1] uint32: device.  An index outside the table gives seg_adv[g] = 0 and sets
 * DRK_STATUS_BAD_SEGMENTS.  S = 0 enqueues nothing.
 */
int drk_segment_advantages(const float* adv, const int32_t* seg_rollout, const int32_t* seg_turn, int32_t R,
                           int32_t Tmax, int32_t S, float* seg_adv, uint32_t* status, void* stream);

/*
 * Reward front-end, upstream of drk_trloo_advantage: per-sample reward and the retention decision of
 * profiling-based rejection sampling.
 *
 *   speedup = min(t_ref / t_kernel, speedup_clip)                      (Sec. 4.2, clip 3)
 *   reward  = C + C * speedup (+ C * PR when use_pr)                    (Eq. 1; profiling reward of Sec. 5.2)
 *   p       = clip((PR - prs_tau) / prs_s, 0, 1)                        (Sec. 5.2, tau = 0.3, s = 0.1)
 *   retain  = 1                          prs_mode = DRK_PRS_OFF
 *             u < p, u ~ U[0,1)          prs_mode = DRK_PRS_SOFT
 *             PR >= prs_tau              prs_mode = DRK_PRS_HARD        (ablation without softness, App. D)
 *
 * u is the top 24 bits, times 2^-24, of the first output word of Philox-4x32-10 (Salmon et al., SC'11)
 * with key = seed (low, high word) and counter = (sample index, offset) (low, high word each): the draw
 * for sample i depends on (seed, offset, i) only.  p and the comparison are taken in fp32.
 * correct [n] uint8 (C = correct != 0), t_ref, t_kernel, pr [n] float, reward [n] float, retain [n] uint8:
 * device.  pr may be NULL when use_pr = 0 and prs_mode = DRK_PRS_OFF; retain may be NULL when
 * prs_mode = DRK_PRS_OFF.  A rejected sample is one the caller leaves out of the loss (clear its
 * loss-mask tokens or give it zero advantage); its reward still enters the group baseline.
 */
typedef enum { DRK_PRS_OFF = 0, DRK_PRS_SOFT = 1, DRK_PRS_HARD = 2 } drk_prs_mode;
typedef struct {
  float speedup_clip; /* default 3 */
  int32_t use_pr;     /* default 0 */
  int32_t prs_mode;   /* drk_prs_mode, default DRK_PRS_OFF */
  float prs_tau;      /* default 0.3 */
  float prs_s;        /* default 0.1 */
  uint64_t seed;      /* default 0 */
  uint64_t offset;    /* default 0; advance per call to draw fresh numbers with one seed */
} drk_reward_params;
void drk_reward_params_default(drk_reward_params* p); /* host pointer */
int drk_reward(const uint8_t* correct, const float* t_ref, const float* t_kernel, const float* pr, int64_t n,
               const drk_reward_params* p, float* reward, uint8_t* retain, void* stream);

/* Parameters of the fused loss.  Fill with drk_pg_params_default() first. */
typedef struct {
  float mrs_lo;          /* Sec. 5.1: retain a sample iff mrs_lo <= w <= mrs_hi; default 0.999       */
  float mrs_hi;          /* default 1.001; mrs_lo <= 0 drops the lower bound, +inf the upper one      */
  float veto_ratio;      /* Sec. 5.1: reject if any token ratio < veto_ratio; default 1e-4; <=0 off   */
  int32_t norm;          /* drk_norm; default DRK_NORM_KEPT_TOKENS                                   */
  float explicit_scale;  /* used when norm == DRK_NORM_EXPLICIT                                      */
  int32_t dw_dtype;      /* drk_dtype of dW; default DRK_F32                                         */
  int32_t dh_dtype;      /* drk_dtype of dH; default DRK_F32                                         */
  int32_t dw_accumulate; /* 0: dW = gradient; 1: dW += gradient (accumulation over micro-batches)    */
  int32_t engine;        /* drk_engine; default DRK_ENGINE_AUTO                                      */
  int32_t v_chunk;       /* vocabulary columns whose dLogits are held at once in the backward;
                            0 = library default (a bf16 buffer of at most 2 GiB: 31232 columns at
                            T = 32768; wider chunks mean fewer passes over the dH accumulator, a
                            smaller value trades a few percent of speed for workspace); rounded up
                            to a multiple of 256                                                    */
  int32_t keep_from_caller; /* 0: seg_keep is an output, decided by MRS here.  1: seg_keep is an INPUT:
                            the caller has already decided which samples are retained (e.g. a sample
                            split over several micro-batches, judged on log-probs from
                            drk_pg_logprob_fwd of all its pieces); seg_w and the counters are still
                            computed from this micro-batch's tokens.  2: seg_keep holds the caller's
                            retention flags on input (for instance `retain` of drk_reward, i.e. the
                            profiling-based rejection sampling of Sec. 5.2) and a sample is kept iff its
                            flag is set AND it passes the MRS test; seg_keep returns the combined decision */
  int32_t forward_rows;  /* 0: log-probs of all T rows.  1: only of the rows the loss can use (loss-masked
                            tokens inside segments); logp, lse, entropy of every other row read 0.  Saves the
                            forward's work on prompt / feedback / padding tokens; tensor-core path only
                            (ignored by the FFMA path)                                                  */
  void* const* dw_chunk_events; /* NULL, or a host array of n_dw_chunk_events cudaEvent_t: event i is recorded
                            on the call's stream as soon as rows [i*vc, min(V,(i+1)*vc)) of dW are final, vc and
                            the chunk count as returned by drk_pg_bwd_chunks().  A data-parallel trainer can
                            wait on them from a communication stream and start reducing finished slices of dW
                            while later chunks are still being computed (the gradient exchange itself is the
                            trainer's; this library makes no collective call)                            */
  int32_t n_dw_chunk_events; /* must equal the chunk count when dw_chunk_events is given                    */
  int32_t reuse_forward; /* 0: the call computes logp, lse (and entropy).  1: logp and lse are INPUTS, as written by
                            an earlier drk_pg_logprob_fwd (or fused call) on the same hidden, W and ids, and the
                            forward pass is skipped: a caller that judged its samples on log-probs from a
                            separate forward (samples split over micro-batches) pays for the logits three times,
                            not four.  entropy is left untouched.  forward_rows must be 0                 */
  int32_t schedule;      /* drk_schedule of the tensor-core kernels' work units; default DRK_SCHEDULE_DYNAMIC.
                            Results are bit-identical either way (every unit's output is independent of
                            which block computes it)                                                     */
} drk_pg_params;

void drk_pg_params_default(drk_pg_params* p); /* host pointer */

/*
 * How the backward of drk_pg_loss_fwd_bwd walks the vocabulary for these sizes: returns the number of
 * chunks (>= 1) and stores the chunk width in *v_chunk (every chunk but the last has that many rows of
 * dW).  Negative drk_status for invalid arguments.  p may be NULL for defaults.
 */
int drk_pg_bwd_chunks(int64_t T, int32_t H, int32_t V, int32_t in_dtype, const drk_pg_params* p,
                      int32_t* v_chunk);

/*
 * Bytes of device workspace needed by drk_pg_logprob_fwd (which = 0) or
 * drk_pg_loss_fwd_bwd (which = 1) for these sizes; p may be NULL for defaults
 * (which = 0 ignores all of p but `engine`).  Returns 0 for invalid arguments.
 * The workspace must be 256-byte aligned.
 */
size_t drk_pg_workspace_bytes(int64_t T, int32_t H, int32_t V, int32_t S, int32_t in_dtype,
                              const drk_pg_params* p, int32_t which);

/*
 * Log-probability of the sampled token under the trainer's LM head, without
 * materialising the logits: the quantity pi_train(a_t | s_t) of Sec. 5.1.
 *
 *   s[t,v]  = sum_h hidden[t,h] * W[v,h]
 *   lse[t]  = log sum_v exp(s[t,v])         (running max / sum over vocabulary tiles)
 *   logp[t] = s[t, ids[t]] - lse[t]
 *
 * hidden [T,H], W [V,H]: device, dtype in_dtype (both the same), 16-byte
 * aligned; for DRK_BF16, H must be a multiple of 8.  ids [T] int32 device.
 * logp, lse [T] float device.  entropy: [T] float device or NULL; when given it
 * receives the entropy of row t's distribution, lse[t] - sum_v p[t,v] s[t,v]
 * (one of the quantities monitored in Sec. 5.1), from the same pass.  status:
 * device uint32, OR-ed into (the caller zeroes it).  engine: drk_engine.
 * T = 0 enqueues nothing.  T <= 2^24, 1 <= V <= 2^24, 1 <= H <= 65536.
 */
int drk_pg_logprob_fwd(const void* hidden, const void* W, int32_t in_dtype, const int32_t* ids,
                       int64_t T, int32_t H, int32_t V, int32_t engine, float* logp, float* lse,
                       float* entropy, void* workspace, size_t workspace_bytes, uint32_t* status,
                       void* stream);

/*
 * The same computation as drk_pg_logprob_fwd for callers that cannot hand over a workspace because they
 * cannot allocate device memory when the call is made: for instance a training loop whose framework
 * already owns all of HBM through its own pool, or a latency-critical section that must avoid
 * cudaMalloc's implicit synchronisation.  (The paper has no counterpart for this entry point; it is a
 * packaging variant of the forward call above.)  The scratch (per-row partial max / sum-exp pairs and
 * target logits) lives in a fixed array inside the library image instead:
 *   - every GPU on which the library is loaded holds DRK_NOALLOC_SCRATCH_BYTES until the process exits;
 *   - if the sizes need more (roughly 16*nsplit*T + 4*T bytes; nsplit, the number of vocabulary ranges per
 *     row tile, is chosen from T and V and is at most 32 for the tensor-core engines and at most 64 for fp32
 *     inputs or DRK_ENGINE_SIMT) the call returns DRK_ERR_WORKSPACE and enqueues nothing; T = 32768 at
 *     H = 5120, V = 151936 needs about 2.2 MB;
 *   - the array is shared by all calls on a device and keeps the last call's contents.  What the
 *     computation reads is rewritten or cleared by each call, so consecutive calls on one stream are
 *     independent; calls that may run concurrently on the GPU (unordered streams) race on it;
 *   - the first call on each device looks up the array's device address.  Make that first call
 *     outside any stream capture.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.  Arguments, outputs, status bits
 * and return codes are those of drk_pg_logprob_fwd, without the workspace pair and without the optional
 * entropy output (this variant returns logp and lse only).
 */
#define DRK_NOALLOC_SCRATCH_BYTES (8u << 20)
int drk_pg_logprob_fwd_noalloc(const void* hidden, const void* W, int32_t in_dtype, const int32_t* ids,
                               int64_t T, int32_t H, int32_t V, int32_t engine, float* logp, float* lse,
                               uint32_t* status, void* stream);

/*
 * Loss and gradients of one packed micro-batch: forward as above, geometric
 * mismatch rejection sampling with token veto per training sample (Sec. 5.1),
 * the REINFORCE surrogate with the caller's per-sample advantages (App. A,
 * with TRLOO advantages per Sec. 4.2), and its gradient with the logits
 * recomputed tile by tile.
 *
 *   segment g     = tokens [cu_seqlens[g], cu_seqlens[g+1]); its masked tokens M_g = {t: loss_mask[t] != 0}
 *   delta_t       = logp[t] - rollout_logp[t]
 *   seg_w[g]      = exp(mean_{t in M_g} delta_t)                  (1 if M_g is empty)
 *   seg_keep[g]   = (ln lo <= mean delta <= ln hi) and (min_{M_g} delta_t >= ln veto) and M_g not empty
 *   c_t           = seg_keep[g(t)] * mask_t * seg_adv[g(t)] * scale      (0 outside every segment)
 *   loss          = - sum_t c_t * logp[t]
 *   dL[t,v]       = c_t * (exp(s[t,v] - lse[t]) - [v == ids[t]])         (c_t is a constant)
 *   dH[t,:]       = sum_v dL[t,v] * W[v,:]       dW[v,:] (+)= sum_t dL[t,v] * hidden[t,:]
 *
 * rollout_logp [T] float, loss_mask [T] uint8, cu_seqlens [S+1] int32
 * (non-decreasing, within [0,T]), seg_adv [S] float: device.  Outputs, all
 * device: loss [1] float; logp, lse [T]; entropy [T] or NULL (as in the forward
 * call); seg_w [S] float; seg_keep [S] uint8;
 * counters [4] int64 = {kept masked tokens, masked tokens in segments, kept
 * segments, vetoed segments}; dH [T,H] of p->dh_dtype; dW [V,H] of
 * p->dw_dtype.  dH and dW must be 16-byte aligned.  With bf16 inputs dL is
 * rounded to bf16 before the two gradient contractions, which accumulate in
 * fp32.  Rows with c_t = 0 get dH = 0 exactly.  S = 0 or T = 0: loss = 0,
 * gradients 0 (dW untouched when accumulating).
 */
int drk_pg_loss_fwd_bwd(const void* hidden, const void* W, int32_t in_dtype, const int32_t* ids,
                        const float* rollout_logp, const uint8_t* loss_mask,
                        const int32_t* cu_seqlens, const float* seg_adv, int64_t T, int32_t H,
                        int32_t V, int32_t S, const drk_pg_params* p, float* loss, float* logp,
                        float* lse, float* entropy, float* seg_w, uint8_t* seg_keep, int64_t* counters,
                        void* dH, void* dW, void* workspace, size_t workspace_bytes, uint32_t* status,
                        void* stream);

/*
 * The same path when the LM head is split by vocabulary rows over several GPUs (each holding rows
 * [v_begin, v_begin + V_local) of W: W_shard is that block, [V_local, H] row-major).  The paper does not
 * say how its trainer lays out the LM head; these two calls compute exactly the quantities defined above
 * (Sec. 5.1 log-probs and rejection, App. A loss and gradient), arranged so that every rank touches only its
 * own rows of W and the ranks exchange two small tensors.  The exchanges are the caller's (this library makes
 * no collective call):
 *
 *   1. every rank:  drk_pg_shard_stats_fwd  ->  stats [T,4] float, per row t over the rank's columns
 *          m = max_v s[t,v]     l = sum_v exp(s[t,v] - m)     r = sum_v exp(s[t,v] - m) * s[t,v]
 *          g = s[t, ids[t]] if v_begin <= ids[t] < v_begin + V_local, else 0
 *   2. all-gather of stats over the ranks  ->  stats_all [n_shards, T, 4] (any order of the ranks)
 *   3. every rank:  drk_pg_shard_loss_bwd   (same arguments as drk_pg_loss_fwd_bwd, plus stats_all)
 *          M = max_k m_k   L = sum_k l_k exp(m_k - M)   lse = M + log L   logp = sum_k g_k - lse
 *          entropy = lse - (sum_k r_k exp(m_k - M)) / L
 *          then rejection sampling, coefficients and loss as in drk_pg_loss_fwd_bwd: loss, logp, lse,
 *          entropy, seg_w, seg_keep and counters come out identical on every rank;
 *          dW_shard [V_local, H] = rows v_begin.. of dW, final;
 *          dH_part [T, H] = sum over the rank's columns of dL[t,v] W[v,:]
 *   4. all-reduce (sum) of dH_part over the ranks = dH.  With more than one rank set p->dh_dtype = DRK_F32 and
 *      convert after the reduction: a part rounded to bf16 first loses bits that the sum would have kept.
 *
 * ids hold token numbers of the whole vocabulary, 0 <= ids[t] < V_total; ids outside set DRK_STATUS_BAD_ID in
 * step 3.  Workspace: drk_pg_workspace_bytes(T, H, V_local, S, in_dtype, p, which) with which = 0 for step 1
 * and 1 for step 3.  p->forward_rows must be 0 in step 3 (DRK_ERR_UNSUPPORTED otherwise).  n_shards <= 4096.
 * stats and stats_all must be 16-byte aligned.  Every other argument, limit, status bit and return code is that
 * of drk_pg_logprob_fwd (step 1) and drk_pg_loss_fwd_bwd (step 3).  With one shard covering the whole
 * vocabulary the results equal those of drk_pg_loss_fwd_bwd.
 */
int drk_pg_shard_stats_fwd(const void* hidden, const void* W_shard, int32_t in_dtype, const int32_t* ids,
                           int64_t T, int32_t H, int32_t V_local, int32_t v_begin, int32_t V_total,
                           int32_t engine, float* stats, void* workspace, size_t workspace_bytes,
                           uint32_t* status, void* stream);
/* Step 3 without loss and gradients: log-probs, lse and (entropy may be NULL) entropy from all ranges'
 * statistics, i.e. drk_pg_logprob_fwd for a vocabulary-split LM head.  All pointers device. */
int drk_pg_shard_merge(const float* stats_all, int32_t n_shards, const int32_t* ids, int64_t T,
                       int32_t V_total, float* logp, float* lse, float* entropy, uint32_t* status,
                       void* stream);
int drk_pg_shard_loss_bwd(const void* hidden, const void* W_shard, int32_t in_dtype, const int32_t* ids,
                          const float* stats_all, int32_t n_shards, const float* rollout_logp,
                          const uint8_t* loss_mask, const int32_t* cu_seqlens, const float* seg_adv,
                          int64_t T, int32_t H, int32_t V_local, int32_t v_begin, int32_t V_total, int32_t S,
                          const drk_pg_params* p, float* loss, float* logp, float* lse, float* entropy,
                          float* seg_w, uint8_t* seg_keep, int64_t* counters, void* dH_part, void* dW_shard,
                          void* workspace, size_t workspace_bytes, uint32_t* status, void* stream);

/*
 * Stability diagnostics of one micro-batch, from the outputs of the calls above: what the paper
 * monitors to diagnose training / inference mismatch (Sec. 5.1, App. B: entropy, perplexity of the
 * trainer and of the rollout engine, gradient norm).  Means run over the loss-masked tokens inside
 * segments.  out: device double[8] =
 *   { n_tokens, mean entropy, exp(-mean logp), exp(-mean rollout_logp), mean (logp - rollout_logp),
 *     max |logp - rollout_logp|, ||dH||_F, ||dW||_F }.
 * entropy, dH, dW may be NULL (their entries are then 0).  dH is [T,H], dW is [V,H] of the given
 * dtypes.  Sums use fp64 atomics: the last digits are not reproducible bit for bit.
 */
int drk_pg_diagnostics(const float* logp, const float* rollout_logp, const float* entropy,
                       const uint8_t* loss_mask, const int32_t* cu_seqlens, int64_t T, int32_t S,
                       const void* dH, int32_t dh_dtype, const void* dW, int32_t dw_dtype, int32_t H,
                       int32_t V, double* out, void* stream);

/*
 * Self-test of the library's failure handling (no counterpart in the paper).  Every on-chip wait of the
 * tensor-core kernels is bounded: when one runs out, the block raises an abort flag that makes its other
 * waiters leave, sets DRK_STATUS_TIMEOUT in the status word and returns, so the context stays usable.  This
 * call launches one block that waits, through the same wait routines, on a barrier that nothing ever signals:
 * one thread with the limit limit_ms (1..1000), one warp with the kernels' own limit (2 s) that must leave
 * early on the abort flag.  Afterwards *status (device, OR-ed into) has DRK_STATUS_TIMEOUT set and waited_ns
 * (device uint64[2]) holds how long the thread and the warp waited.  Nothing else is touched.
 */
int drk_selftest_bounded_wait(uint32_t limit_ms, uint32_t* status, uint64_t* waited_ns, void* stream);

/* Number of kernels the last call on this host thread enqueued (0 after an error). */
int drk_last_launch_count(void);

/*
 * Number of TMA tensor maps this process has encoded so far (no counterpart in the paper).  Maps depend on a
 * buffer's address and geometry only and are cached, so a call that repeats an earlier call's pointers and
 * sizes (the steady state of a training loop) adds nothing to this count.
 */
uint64_t drk_tensor_map_encodes(void);

/*
 * Host-side fault injection for tests of the error contract (no counterpart in the paper): the nth next request
 * for a tensor map inside this process fails as if the driver had refused to encode it (nth >= 1; 0 clears a
 * pending injection).  The call that hits it returns DRK_ERR_CUDA, and because all maps are built before the
 * first enqueue it must leave the stream and every output untouched.  Nothing on the device is made to fail.
 */
void drk_selftest_fail_tensor_map(int32_t nth);

const char* drk_status_string(int status);
int drk_version(void);
/* 1 if this library was compiled with -DDRK_BOUNDS_CHECK (see DRK_STATUS_BOUNDS), else 0. */
int drk_bounds_checked(void);

#ifdef __cplusplus
}
#endif
#endif /* DRK_H_ */
