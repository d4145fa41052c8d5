/*
 * cocodc.h - C ABI of the CoCoDC outer synchronisation step for NVIDIA B200 (sm_100a).
 *
 * The library implements what CoCoDC ("Cross-region Model Training with
 * Communication-Computation Overlapping and Delay Compensation") does to
 * parameter memory when the synchronisation of a model fragment completes, and
 * the decision which fragments to synchronise next:
 *
 *   S0  record theta^m_{p,t_p} when a sync is initiated           (Algorithm 1, input)
 *   S1  per-worker pseudo-gradient  theta^m_{p,t_p} - theta^g_{p,t_p-H}   (Section 2.1)
 *   S2  their mean over the M workers                              (Eq. 1)
 *   S3  outer optimizer: SGD with Nesterov momentum                (Eq. 2)
 *   S4  Taylor-expansion delay compensation                        (Eq. 4-7, Algorithm 1)
 *   S5  merge into every worker's local parameters                 (Eq. 7 / Eq. 3)
 *   S6  per-fragment change-rate score R_p = ||Delta theta^g_p|| / I_p   (Eq. 10)
 *   S7  fragment selection under a budget                          (Algorithm 2, Eq. 11)
 *   S8  schedule sizing N, h                                       (Eq. 8-9)
 *
 * The M workers are M stacked replicas in one GPU's memory; the mean over
 * workers is a reduction along that axis, not a collective.
 *
 * Conventions
 *   - "dev" pointers are device-memory addresses, "host" pointers host addresses.
 *     All parameter data is fp32.  Streams are passed as void* (a cudaStream_t;
 *     NULL is the default stream).
 *   - The caller owns every buffer it passes.  The library owns only the context
 *     (a copy of the fragment table, a few KB of launch scratch, a status word),
 *     allocated by cocodc_create and released by cocodc_destroy.
 *   - Device entry points are asynchronous on the given stream and allocate
 *     nothing, neither device nor host memory.  Their return value reports host-side validation and launch
 *     errors; conditions found on the device (a non-finite norm, an invalid id
 *     list, a NaN score) are recorded in the context's status word, read with
 *     cocodc_poll_status.  Nothing aborts, traps or prints.
 *   - Base pointers of parameter buffers must be 16-byte aligned and row strides
 *     multiples of 4 elements (COCODC_ERR_ALIGNMENT otherwise).  Segment offsets
 *     and lengths are arbitrary; ragged edges are handled inside the kernels.
 *   - Offsets, strides and sizes are int64 (element counts): M*N exceeds 2^32 for
 *     billion-parameter models.
 *   - A context serialises its own launches on one stream at a time: calls that
 *     share a context must not overlap on the GPU.
 *   - Step numbers (t_now, t_p, t_l, last_sync[p]) are non-negative and last_sync[p] <= t_now, t_p:
 *     differences of step numbers are formed in 64-bit integers and must not overflow.
 *   - Every wait inside a kernel is bounded.  A launch whose wait ran out records COCODC_ERR_TIMEOUT
 *     and returns early; its outputs, and those of later launches on the stream, are undefined until
 *     the caller has read the status (cocodc_poll_status synchronises and resets the context).
 */
#ifndef COCODC_H
#define COCODC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  COCODC_OK = 0,
  COCODC_ERR_INVALID_ARG = 1,
  COCODC_ERR_ALIGNMENT = 2,
  COCODC_ERR_ALIAS = 3,
  COCODC_ERR_NONFINITE = 4,   /* device: a fragment norm or a score was NaN/Inf where not allowed */
  COCODC_ERR_TIMEOUT = 5,     /* device: a bounded wait ran out */
  COCODC_ERR_CUDA = 6,
  COCODC_ERR_NOMEM = 7
} cocodc_status;

/* How the merged local parameters are formed (S4-S5). */
typedef enum {
  COCODC_COMP_NONE = 0,    /* no compensation: blend the new global state, Eq. 3 (Streaming DiLoCo, DiLoCo) */
  COCODC_COMP_TAYLOR = 1   /* Eq. 4-7 */
} cocodc_comp_mode;

/*
 * Eq. 4 as printed takes theta_{t_p} - theta_{t_l} while the text calls it the
 * change rate over the overlap and Eq. 7 adds it; the three consistent readings
 * are all available.  With d = a - b (a = theta^m_{t_l}, b = theta^m_{t_p}),
 * D = G - b, G = theta^g_{p,t_p}, c = lambda/(tau*H):
 *   FORWARD : target = G + d + c*d*d*D   (rate taken forward in time; default)
 *   PRINTED : target = G - d + c*d*d*D   (Eq. 4, 6, 7 literally)
 *   DESCENT : target = G + d - c*d*d*D   (Eq. 4-6 literally, Eq. 7 subtracting)
 */
typedef enum {
  COCODC_SIGN_FORWARD = 0,
  COCODC_SIGN_PRINTED = 1,
  COCODC_SIGN_DESCENT = 2
} cocodc_sign_mode;

/* COUNT and PARAMS walk the priority order greedily; PARAMS_EXACT (an option the paper does not have)
 * solves the parameter budget as a knapsack, see cocodc_select_fragments. */
typedef enum { COCODC_BUDGET_COUNT = 0, COCODC_BUDGET_PARAMS = 1, COCODC_BUDGET_PARAMS_EXACT = 2 } cocodc_budget_kind;
#define COCODC_EXACT_MAX_CANDIDATES 24

/* Stages of cocodc_outer_step. */
#define COCODC_STAGE_OUTER 1u   /* S1-S3: update theta_g and momentum (required) */
#define COCODC_STAGE_MERGE 2u   /* S4-S5: update w_now */
#define COCODC_STAGE_SCORE 4u   /* S6: norms, scores, last_sync of the processed fragments */
#define COCODC_STAGE_ALL   7u
#define COCODC_STAGE_SUMSQ 8u   /* S6 up to the sums only: sumsq_out[p] = sum of Delta^2 over fragment p (Eq. 10 before the
                                   square root), for callers that add the sums of several devices before forming scores */
#define COCODC_STAGE_DEFER 16u  /* with COCODC_STAGE_SCORE (and without sumsq_out): the launch ends once every thread block
                                   has left its sum of squares per fragment in the context's scratch; the square root, the
                                   division by I_p, last_sync and the in-flight marks (the rest of Eq. 10 and the text after
                                   it) are formed by the next call on the context that decides on fragments -
                                   cocodc_initiate(_at), in the prologue of its one launch when it is given the same scores
                                   and last_sync arrays - or, failing that, by one small launch placed before any other
                                   call that reads or writes norms, scores, last_sync or that scratch (cocodc_outer_step
                                   and its variants, cocodc_select_fragments(_at), cocodc_fragment_scores,
                                   cocodc_scores_from_sumsq, cocodc_outer_step_host) or by cocodc_flush_scores.  Until
                                   then norms, scores, last_sync and the in-flight marks keep their previous contents.
                                   The values are bit for bit those of the undeferred stage.  Why: forming the scores
                                   inside the completion's launch costs a grid-wide hand-off after its last tile (about
                                   7 us whatever the launch size); the boundary to the next launch is that hand-off. */

/*
 * Fragment partition (Section 2.1: the model is cut into K disjoint fragments).
 * CSR over segments: fragment p owns segments frag_seg_ptr[p] .. frag_seg_ptr[p+1]-1,
 * each a run of seg_len[s] elements starting at element seg_offset[s] of every
 * N-sized buffer.  A strided shard (Section 4.1) is a fragment with several
 * segments.  Segments must not overlap and must lie inside [0, N).  All three
 * arrays are host memory and are copied by cocodc_create.
 */
typedef struct {
  int64_t N;
  int32_t K;
  int32_t n_segments;
  const int32_t* frag_seg_ptr;  /* host, K+1 */
  const int64_t* seg_offset;    /* host, n_segments */
  const int64_t* seg_len;       /* host, n_segments */
} cocodc_partition;

/* Hyper-parameters of one completion (paper symbols in brackets). */
typedef struct {
  int32_t M;          /* worker replicas [M], 1..64 */
  int32_t comp_mode;  /* cocodc_comp_mode */
  int32_t sign_mode;  /* cocodc_sign_mode */
  int32_t reserved;
  int64_t H;          /* local steps between syncs of a fragment [H], > 0 */
  int64_t tau;        /* overlap depth [tau], >= 0; 0 only with COMP_NONE or w_snap == w_now */
  float outer_lr;     /* outer learning rate (Eq. 2) */
  float momentum;     /* outer Nesterov momentum (Eq. 2) */
  float lambda;       /* compensation strength [lambda] (Eq. 6) */
  float alpha;        /* mixing factor [alpha] (Eq. 3); 1 assigns the target (Eq. 7) */
} cocodc_hyper;

typedef struct cocodc_ctx cocodc_ctx;

/*
 * Create a context for one partition on one device.  max_M bounds hyper.M of
 * later calls.  Allocates device scratch (cudaMalloc) and copies the fragment
 * table.  Errors: INVALID_ARG (NULLs, K < 1, K > 1024, overlapping or
 * out-of-range segments, empty fragments, max_M outside 1..64), NOMEM, CUDA.
 */
cocodc_status cocodc_create(cocodc_ctx** ctx_out, const cocodc_partition* partition,
                            int32_t max_M, int32_t device);
cocodc_status cocodc_destroy(cocodc_ctx* ctx);

/*
 * S8, host only.  Eq. 8: N = max(K, floor(gamma*H*Tc/Ts)); Eq. 9: h = floor(H/N),
 * raised to 1 when N > H.  Tc, Ts: seconds per local step / per fragment sync.
 * INVALID_ARG unless K >= 1, H >= 1, 0 < gamma <= 1, Tc > 0, Ts > 0.
 */
cocodc_status cocodc_sync_budget(int32_t K, int64_t H, double gamma, double Tc, double Ts,
                                 int64_t* N_out, int64_t* h_out);

/*
 * S6 stand-alone (Eq. 10): norms[p] = ||delta_g restricted to fragment p||_2 and
 * scores[p] = norms[p] / max(1, interval[p]) for all K fragments.
 *   delta_g  dev fp32[N]   the received mean pseudo-gradients
 *   interval dev int64[K]  I_p = t_p - t_{p,b}; NULL means 1
 *   norms, scores dev fp32[K], written (both NULL: only sumsq_out is wanted)
 *   sumsq_out dev fp64[K] or NULL: the sums of squares before the square root
 * Sums of squares are accumulated in double in a fixed order (run-to-run
 * reproducible).  A non-finite norm sets COCODC_ERR_NONFINITE in the status word.
 * One kernel launch: the last warp to finish forms the norms.
 */
cocodc_status cocodc_fragment_scores(cocodc_ctx* ctx, const float* delta_g, const int64_t* interval,
                                     float* norms, float* scores, double* sumsq_out, void* stream);

/*
 * The rest of Eq. 10 from sums of squares that already exist: when every device holds a slice of each
 * fragment (all workers of an element range), a fragment's norm spans devices; each device takes its sums
 * from cocodc_outer_step (COCODC_STAGE_SUMSQ) or cocodc_fragment_scores (sumsq_out), the caller adds them
 * over the devices (an all-reduce of K doubles), and this call forms norms and scores from the totals:
 *   norms[p] = sqrt(sumsq[p]),  scores[p] = norms[p] / max(1, I_p)
 *   sumsq dev fp64[K], indexed by fragment id
 *   completion (ids, n_ids given; interval NULL): for the listed fragments I_p = t_p - last_sync[p], then
 *       last_sync[p] = t_l (and a bound in-flight mask is cleared, see cocodc_bind_in_flight)
 *   stand-alone (ids, n_ids NULL): all K fragments, I_p = interval[p] (1 without intervals); t_p, t_l and
 *       last_sync are not used
 * A non-finite norm sets COCODC_ERR_NONFINITE, an id outside [0, K) INVALID_ARG, in the status word.
 */
cocodc_status cocodc_scores_from_sumsq(cocodc_ctx* ctx, const double* sumsq, const int32_t* ids, const int32_t* n_ids,
                                       const int64_t* interval, int64_t t_p, int64_t t_l, int64_t* last_sync,
                                       float* norms, float* scores, void* stream);

/*
 * Algorithm 2's bookkeeping of the fragments whose synchronisation is in flight (a fragment chosen at t_p
 * cannot be chosen again before it completes at t_p + tau).  in_flight is a dev uint8[K] array owned by the
 * caller, zero-initialised by it; once bound to the context,
 *   cocodc_select_fragments(_at) and cocodc_initiate treat in_flight[p] != 0 as not eligible and set
 *                                 in_flight[p] = 1 for every fragment they select,
 *   every completion that writes scores (cocodc_outer_step and its variants with COCODC_STAGE_SCORE,
 *   cocodc_scores_from_sumsq with an id list) sets in_flight[p] = 0 for the fragments it lists.
 * NULL unbinds.  The host-buffer entry points do not use it.
 */
cocodc_status cocodc_bind_in_flight(cocodc_ctx* ctx, uint8_t* in_flight);

/*
 * Forms the norms, scores, last_sync entries and in-flight marks that a completion launched with
 * COCODC_STAGE_DEFER has left unformed (one launch of one thread block on `stream`, which must be the
 * stream of that completion or ordered after it); does nothing when no such completion is outstanding.
 * The arrays written are the ones that completion was given.  Errors: INVALID_ARG for a NULL context; a
 * non-finite norm is reported through the status word (COCODC_ERR_NONFINITE) as in the undeferred stage.
 */
cocodc_status cocodc_flush_scores(cocodc_ctx* ctx, void* stream);

/*
 * S7 (Algorithm 2, Eq. 11, extended to a budget).  Priority order: eligible
 * fragments with t_now - last_sync[p] >= H by ascending index (Algorithm 2's
 * loop), then the other eligible fragments by score, largest first, ties to the
 * lower index; +Inf is a legal score (never-synced fragments).  The head of the
 * order is always taken; each later fragment is taken iff its cost (1 for
 * COUNT, its size for PARAMS) still fits what is left of the budget.  budget = 1
 * (COUNT) is exactly Algorithm 2.
 *   scores dev fp32[K]; last_sync dev int64[K]; ineligible dev uint8[K] or NULL
 *   mask dev uint8[K] (1 = selected); ids dev int32[K] (first n_sel entries, admission
 *   order; the rest set to -1); n_sel dev int32[1]
 *   pool_offset dev int64[K] or NULL: if given, the selected fragments are assigned places in a
 *   packed snapshot pool (the snap_offset argument of the calls below): admission order, back to
 *   back, each start at the next multiple of 4 elements plus (native offset of the fragment's
 *   first segment) mod 4, so that recorded and native values share their 16-byte alignment and
 *   the streaming calls move the fragment as vectors; -1 for fragments not selected.  A pool row
 *   of budget + (largest fragment) elements (PARAMS), or the `budget` largest fragments (COUNT),
 *   plus 8 per fragment for alignment, always suffices.  (Callers that place fragments themselves
 *   should keep the same congruence: a segment whose pool position differs from its native offset
 *   by a non-multiple of 4 cannot be staged by bulk copies and runs at half to two thirds of the bandwidth.)
 * A NaN score selects nothing and sets COCODC_ERR_NONFINITE.
 *
 * PARAMS_EXACT (no counterpart in the paper, whose Algorithm 2 picks one fragment per decision): the
 * fragments that must go first -- the overdue ones and those with score +Inf -- are walked as for PARAMS;
 * among the remaining eligible fragments the subset with the largest sum of scores whose sizes fit what is
 * left of the budget is taken (sum formed in double in priority order; equal sums go to the subset that,
 * written as a bit string over the priority order with the first fragment as lowest bit, is the smaller
 * number).  If nothing was taken at all, the first fragment of the order is (a decision always returns one).
 * ids lists the forced fragments first, then the subset in priority order.  At most
 * COCODC_EXACT_MAX_CANDIDATES fragments may remain for the subset search (it enumerates all subsets); more
 * selects nothing and sets COCODC_ERR_INVALID_ARG in the status word.
 */
cocodc_status cocodc_select_fragments(cocodc_ctx* ctx, const float* scores, const int64_t* last_sync,
                                      const uint8_t* ineligible, int64_t t_now, int64_t H,
                                      int32_t budget_kind, int64_t budget,
                                      uint8_t* mask, int32_t* ids, int32_t* n_sel,
                                      int64_t* pool_offset, void* stream);

/*
 * S1-S6 fused, at completion time t_l, for the fragments listed on the device
 * (typically the ids that cocodc_select_fragments wrote tau steps earlier).
 * Per element i of each listed fragment, in fp32:
 *   Delta = (sum_m (w_snap[m][i] - theta_g[i])) / M                        (Eq. 1)
 *   u'    = momentum*u + Delta ; G = theta_g + outer_lr*(Delta + momentum*u')   (Eq. 2)
 *   target_m = per sign_mode above, or G for COMP_NONE                     (Eq. 4-7)
 *   w_now[m][i] = (1-alpha)*w_now[m][i] + alpha*target_m                   (Eq. 3 / Eq. 7)
 * and theta_g[i] = G, momentum[i] = u', delta_g_out[i] = Delta (if not NULL).
 * With STAGE_SCORE, for each listed p: norms[p] = ||Delta||_2 over the fragment,
 * scores[p] = norms[p] / max(1, t_p - last_sync[p]), then last_sync[p] = t_l.
 * With STAGE_SUMSQ (or STAGE_SCORE and sumsq_out not NULL): sumsq_out[p] = sum of Delta^2 over the fragment.
 * Fragments not listed are not touched.  The whole call is one kernel launch (the id list is expanded by
 * the kernel itself and the norms are formed by its last warp) for fragment tables of up to 128 segments;
 * larger tables take one more small launch.
 *
 *   w_now   dev fp32, worker m's element i at w_now[m*now_stride + i]   (theta^m_{.,t_l}, in/out)
 *   w_snap  dev fp32, theta^m_{p,t_p}: at w_snap[m*snap_stride + i] if snap_offset is NULL,
 *           else fragment p packed (segments back to back) from w_snap[m*snap_stride + snap_offset[p]]
 *           w_snap == w_now (same stride, snap_offset NULL) is legal: zero delay, blocking sync
 *   snap_offset dev int64[K] or NULL
 *   theta_g, momentum dev fp32[N] in/out; delta_g_out dev fp32[N] or NULL
 *   ids dev int32[<=K] distinct fragment ids; n_ids dev int32[1]
 *   last_sync dev int64[K]; norms, scores dev fp32[K] (needed with STAGE_SCORE)
 *   sumsq_out dev fp64[K] (needed with STAGE_SUMSQ), or NULL
 * Errors: INVALID_ARG, ALIGNMENT, ALIAS (buffers overlapping other than w_snap == w_now), CUDA.
 * Device-side: an id outside [0,K) or listed twice, a listed fragment without a place in the pool
 * (snap_offset[p] < 0) or whose packed snapshot would not fit inside one row (snap_offset[p] + n_p >
 * snap_stride) processes nothing and sets INVALID_ARG.
 */
cocodc_status cocodc_outer_step(cocodc_ctx* ctx, const cocodc_hyper* hyper,
                                float* w_now, const float* w_snap,
                                int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                float* theta_g, float* momentum, float* delta_g_out,
                                const int32_t* ids, const int32_t* n_ids,
                                int64_t t_p, int64_t t_l, int64_t* last_sync,
                                float* norms, float* scores, double* sumsq_out, uint32_t stages, void* stream);

/*
 * cocodc_select_fragments and cocodc_outer_step with their step numbers read from DEVICE memory at run time
 * (t_now, t_p, t_l: dev int64[1] each) instead of passed by value.  Everything else is identical.  A schedule
 * step (completion, selection, snapshot) contains no host-side value that changes from step to step any more,
 * so it can be recorded once in a CUDA graph and replayed while a device-side counter advances - which is
 * what makes small workloads, whose step is a handful of microsecond kernels, launch-bound no longer.
 */
cocodc_status cocodc_select_fragments_at(cocodc_ctx* ctx, const float* scores, const int64_t* last_sync,
                                         const uint8_t* ineligible, const int64_t* t_now, int64_t H,
                                         int32_t budget_kind, int64_t budget,
                                         uint8_t* mask, int32_t* ids, int32_t* n_sel,
                                         int64_t* pool_offset, void* stream);
cocodc_status cocodc_outer_step_at(cocodc_ctx* ctx, const cocodc_hyper* hyper,
                                   float* w_now, const float* w_snap,
                                   int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                   float* theta_g, float* momentum, float* delta_g_out,
                                   const int32_t* ids, const int32_t* n_ids,
                                   const int64_t* t_p, const int64_t* t_l, int64_t* last_sync,
                                   float* norms, float* scores, double* sumsq_out, uint32_t stages, void* stream);

/*
 * Worker-per-device deployment (Section 2.1: every worker all-reduces its pseudo-gradient).  When a
 * device holds only M of the M_total workers, Eq. 1's sum spans devices:
 *
 *   cocodc_pseudo_gradient_sum   S1 + the local part of S2: sum_out[i] = sum over this device's M
 *                                workers of (w_snap[m][i] - theta_g[i]) for the listed fragments, at their
 *                                native offsets in sum_out (dev fp32[N]); other elements are not touched.
 *   (the caller all-reduces sum_out over the devices, e.g. with NCCL)
 *   cocodc_outer_step_received   S2-S6 as cocodc_outer_step (all stages), except that
 *                                Delta = delta_sum[i] / M_total; hyper->M is the local worker count, whose
 *                                w_now rows are merged.  delta_g_out may be NULL, or delta_sum itself
 *                                (replaced by Delta in place).
 *
 * With M_total == hyper->M and delta_sum produced by cocodc_pseudo_gradient_sum on the same buffers the
 * result is bit-identical to cocodc_outer_step.  Layout, alignment and device-side error rules as there;
 * w_snap == w_now (zero delay) is not accepted here.
 */
cocodc_status cocodc_pseudo_gradient_sum(cocodc_ctx* ctx, const float* w_snap, int64_t snap_stride,
                                         const int64_t* snap_offset, const float* theta_g, int32_t M,
                                         float* sum_out, const int32_t* ids, const int32_t* n_ids, void* stream);
cocodc_status cocodc_outer_step_received(cocodc_ctx* ctx, const cocodc_hyper* hyper, int32_t M_total,
                                         float* w_now, const float* w_snap,
                                         int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                         float* theta_g, float* momentum, const float* delta_sum,
                                         float* delta_g_out, const int32_t* ids, const int32_t* n_ids,
                                         int64_t t_p, int64_t t_l, int64_t* last_sync,
                                         float* norms, float* scores, void* stream);

/*
 * The same step with the exchange of Section 2.1 folded in: instead of one all-reduced buffer the call takes
 * the n_sums (1..COCODC_MAX_SUMS) buffers that cocodc_pseudo_gradient_sum wrote on the contributing devices
 * and adds them itself, in the listed order, while it streams the fragment:
 *   Delta = (delta_sums[0][i] + delta_sums[1][i] + ... ) / M_total      (fp32, left to right)
 * so the summed pseudo-gradient is never written to or re-read from memory.  delta_sums is a HOST array of
 * device pointers (dev fp32[N] each, 16-byte aligned); entries may point into other devices' memory that is
 * mapped into this process (peer access, CUDA IPC or a symmetric-memory allocation): the kernel reads them
 * with ordinary one-CTA bulk copies (no cluster-wide form), each element once.  Every device that lists the buffers in the same
 * order computes bit-identical Delta, theta_g and momentum.  The caller orders the calls across devices: all
 * cocodc_pseudo_gradient_sum calls must have completed before any device starts this call, and no buffer may
 * be overwritten until every device has finished it (a barrier on the host, or stream events, before and
 * after).  delta_g_out may be NULL or one of the listed buffers of THIS device (replaced by Delta in place).
 * With n_sums == 1 this is cocodc_outer_step_received.
 * Reads from another device's memory have not been exercised on hardware: every test so far passed buffers of
 * the calling device.
 */
#define COCODC_MAX_SUMS 8
cocodc_status cocodc_outer_step_received_peers(cocodc_ctx* ctx, const cocodc_hyper* hyper, int32_t M_total,
                                               float* w_now, const float* w_snap,
                                               int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                               float* theta_g, float* momentum,
                                               const float* const* delta_sums, int32_t n_sums,
                                               float* delta_g_out, const int32_t* ids, const int32_t* n_ids,
                                               int64_t t_p, int64_t t_l, int64_t* last_sync,
                                               float* norms, float* scores, void* stream);

/*
 * S4-S5 alone (Algorithm 1, or Eq. 3 for COMP_NONE), given the new global state:
 * w_now[m][i] = (1-alpha)*w_now[m][i] + alpha*target_m with G = theta_g_new[i].
 * Together with cocodc_outer_step(stages without MERGE) this is the unfused path.
 */
cocodc_status cocodc_merge(cocodc_ctx* ctx, const cocodc_hyper* hyper,
                           float* w_now, const float* w_snap,
                           int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                           const float* theta_g_new, const int32_t* ids, const int32_t* n_ids,
                           void* stream);

/*
 * S0: copy the listed fragments of every worker from w_now into w_snap (same
 * layout rules as above) when their synchronisation is initiated at t_p.
 */
cocodc_status cocodc_snapshot(cocodc_ctx* ctx, const float* w_now, float* w_snap,
                              int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                              int32_t M, const int32_t* ids, const int32_t* n_ids, void* stream);

/*
 * Initiation of a synchronisation at t_p in one call: Algorithm 2 (as cocodc_select_fragments, same arguments
 * and outputs) followed by S0 for the fragments it picked (as cocodc_snapshot, with the places just written to
 * pool_offset as the snapshot layout; pool_offset NULL keeps the native layout).  The two always happen
 * together in the method - a fragment is chosen and its theta^m_{p,t_p} recorded - and for fragment tables of
 * up to 128 segments and the COUNT and PARAMS budgets they are ONE kernel launch: every block of the snapshot
 * kernel works out the (deterministic) selection for itself in its prologue.  Larger tables and
 * COCODC_BUDGET_PARAMS_EXACT run the two kernels one after the other.  Results are bit-identical to the two
 * separate calls.  The output arrays (mask, ids, n_sel, pool_offset) must not overlap the inputs.
 */
cocodc_status cocodc_initiate(cocodc_ctx* ctx, const float* scores, const int64_t* last_sync,
                              const uint8_t* ineligible, int64_t t_now, int64_t H,
                              int32_t budget_kind, int64_t budget,
                              uint8_t* mask, int32_t* ids, int32_t* n_sel, int64_t* pool_offset,
                              const float* w_now, float* w_snap, int64_t now_stride, int64_t snap_stride, int32_t M,
                              void* stream);

/* cocodc_initiate with t_now read from device memory (dev int64[1]) at run time, for graph replay (see
 * cocodc_select_fragments_at). */
cocodc_status cocodc_initiate_at(cocodc_ctx* ctx, const float* scores, const int64_t* last_sync,
                                 const uint8_t* ineligible, const int64_t* t_now, int64_t H,
                                 int32_t budget_kind, int64_t budget,
                                 uint8_t* mask, int32_t* ids, int32_t* n_sel, int64_t* pool_offset,
                                 const float* w_now, float* w_snap, int64_t now_stride, int64_t snap_stride, int32_t M,
                                 void* stream);

/*
 * S1-S6 as cocodc_outer_step (all stages), for callers whose parameters live in HOST memory.
 * Every buffer argument here is a host pointer (pinned memory makes the copies asynchronous and
 * fast; pageable memory works); ids is a host array of n_ids fragment ids; last_sync, norms and
 * scores are host arrays of K entries, updated for the listed fragments.  The listed fragments
 * are streamed through the device in chunks: host->device copies, the fused kernel and
 * device->host copies of consecutive chunks overlap on three streams.  Results are in host
 * memory when the call returns (it synchronises).  Host pointers need no particular alignment.
 *   snap_on_device   0: w_snap is a host buffer like the others.  1: w_snap (and only it) is DEVICE
 *                    memory, e.g. a snapshot pool filled by cocodc_snapshot_host at t_p, read in place
 *                    (16-byte aligned, stride a multiple of 4); snap_offset stays a host array
 *   workspace        dev, 16-byte aligned staging memory provided by the caller
 *   workspace_bytes  at least 3*(2M+3)*4096*4 bytes; a few hundred MB gives full-size chunks
 *   stream           the stream the kernels run on (two internal streams carry the copies)
 * Sums of squares are accumulated chunk by chunk in a fixed order.
 */
cocodc_status cocodc_outer_step_host(cocodc_ctx* ctx, const cocodc_hyper* hyper,
                                     float* w_now, const float* w_snap,
                                     int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                     float* theta_g, float* momentum, float* delta_g_out,
                                     const int32_t* ids, int32_t n_ids,
                                     int64_t t_p, int64_t t_l, int64_t* last_sync,
                                     float* norms, float* scores, int32_t snap_on_device,
                                     void* workspace, uint64_t workspace_bytes, void* stream);

/*
 * S0 for parameters that live in host memory: copy the listed fragments of every worker from the
 * HOST buffer w_now into the DEVICE buffer w_snap (layout rules as for cocodc_snapshot; ids and
 * snap_offset are host arrays).  Asynchronous on the stream when w_now is pinned.  The snapshot
 * then waits on the device for the completion tau steps later (cocodc_outer_step_host with
 * snap_on_device = 1), so it crosses the bus once.
 */
cocodc_status cocodc_snapshot_host(cocodc_ctx* ctx, const float* w_now, float* w_snap,
                                   int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                   int32_t M, const int32_t* ids, int32_t n_ids, void* stream);

/*
 * (No counterpart in the paper: this is an interface variant, not a step of the method.)
 * cocodc_fragment_scores for callers that cannot allocate device memory - code running inside an
 * allocator hook or a memory-pool callback, processes whose device memory is handed out up front
 * and whose runtime heap is closed, latency-critical paths that must not hit an allocation's
 * implicit synchronisation.  Such callers cannot use cocodc_create either, so the fragment table
 * is passed directly (host arrays, validated on every call) and no context is involved.
 *
 * Same result as cocodc_fragment_scores: norms[p] = ||delta_g restricted to fragment p||_2,
 * scores[p] = norms[p] / max(1, interval[p]) (interval NULL means 1).  A non-finite norm is
 * written as it is; there is no status word.
 *
 * The scratch (per-CTA partial sums, about 0.6 MB) is a fixed __device__ array inside the library
 * image: every GPU that loads the library holds it until the process exits.  Its size bounds the
 * problem: K <= COCODC_NOALLOC_MAX_K fragments and n_segments <= COCODC_NOALLOC_MAX_SEGMENTS;
 * anything larger returns COCODC_ERR_INVALID_ARG.  The call itself makes no cudaMalloc/cudaFree
 * and calls no allocating library routine; it launches two kernels on `stream`.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with that
 * device current) and caches it; make that first call outside any stream capture.
 * All calls on a device share the one array: each call rewrites every entry it later reads, so the
 * previous call's contents never matter, but two calls that overlap on the GPU (different streams,
 * different threads) race on it - serialise them.
 *   partition  host; delta_g dev fp32[N], 16-byte aligned; interval dev int64[K] or NULL;
 *   norms, scores dev fp32[K]; device = the CUDA device the pointers belong to
 */
#define COCODC_NOALLOC_MAX_K 64
#define COCODC_NOALLOC_MAX_SEGMENTS 64
cocodc_status cocodc_fragment_scores_noalloc(const cocodc_partition* partition, const float* delta_g,
                                             const int64_t* interval, float* norms, float* scores,
                                             int32_t device, void* stream);

/*
 * Waits for the stream, then returns and clears the device status word
 * (COCODC_OK if nothing was recorded since the last poll).  After an error the context's launch
 * scratch is reset, so the next call starts clean; a completion launched with COCODC_STAGE_DEFER whose
 * scores have not been formed by then is dropped with it (its outputs are undefined after the error, as
 * those of every launch before the poll).
 */
cocodc_status cocodc_poll_status(cocodc_ctx* ctx, void* stream);

/*
 * Failure-detection self-test.  The staged kernels wait on shared-memory barriers for their bulk
 * copies; every such wait gives up after a fixed number of polls, records COCODC_ERR_TIMEOUT in the
 * status word and lets the kernel return (a producer first waits, again with a limit, for the copies
 * it has already started, so that they do not land in shared memory that has moved on to another block).
 * This call runs that wait on a barrier nothing will complete, with `polls` (1 .. 4194304) as the limit:
 * afterwards cocodc_poll_status returns COCODC_ERR_TIMEOUT and the context is as usable as before.  It
 * cannot hang: the loop is bounded.
 */
cocodc_status cocodc_selftest_bounded_wait(cocodc_ctx* ctx, int32_t polls, void* stream);

/* Number of kernels the library has launched through this context so far. */
int64_t cocodc_launch_count(const cocodc_ctx* ctx);

const char* cocodc_status_string(cocodc_status s);

#ifdef __cplusplus
}
#endif
#endif /* COCODC_H */
