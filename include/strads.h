/*
 * strads.h -- C ABI of the B200 scheduled-Lasso library (libstrads_b200.so).
 *
 * One scheduled round of parallel coordinate descent for the Lasso, after
 * Lee, Kim, Ho, Gibson, Xing, "Structure-Aware Dynamic Scheduler for Parallel
 * Machine Learning" (Section 2, SAP steps 1-4; Section 2.1, Algorithm 1, Eq. 1,
 * Eq. 2; Section 4, Theorem 1 for the sampling weight).
 *
 * Notation (the paper's): X is N x J with standardised columns x_j, y has N
 * entries, beta has J; P' candidates are drawn per round (n_candidates), at
 * most P of them are updated in parallel (n_keep); eta, rho, lambda as in
 * Algorithm 1; delta_j = |beta_j^(t_j-1) - beta_j^(t_j-2)| is the stored last
 * change of coefficient j and starts at the "very large constant" C (c_init).
 *
 * Conventions for every call
 *   - plain C, no exceptions; returns STRADS_OK (0) or a negative strads_status_t;
 *   - "device" pointers are CUDA device addresses on the device that was current
 *     at strads_lasso_init; "host" pointers are ordinary host addresses;
 *   - every array is allocated, owned and freed by the caller; the handle owns
 *     only host bookkeeping.  X and y are never written and must outlive the
 *     handle, as must beta, resid, delta and the workspace;
 *   - the library allocates no device memory (strads_sample_static keeps about 65 KB of scratch in a
 *     fixed device array of its own instead of a workspace);
 *   - arguments are validated on the host before anything is launched; nothing
 *     traps, aborts or waits without a bound;
 *   - calls are asynchronous on the configured stream unless stated otherwise;
 *   - one handle <-> one stream <-> one host thread at a time;
 *   - same inputs, seed and round index give bit-identical outputs (no
 *     floating-point atomics anywhere).
 */
#ifndef STRADS_H_
#define STRADS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct strads_lasso_s* strads_handle_t;   /* opaque host object */

typedef enum {
  STRADS_OK = 0,
  STRADS_ERR_INVALID_ARG = -1,          /* NULL / out-of-range / misaligned argument          */
  STRADS_ERR_BAD_LAYOUT = -2,           /* unknown layout, ld too small or not a multiple of 4 */
  STRADS_ERR_WORKSPACE_TOO_SMALL = -3,
  STRADS_ERR_CUDA = -4,                 /* a CUDA runtime call failed (see strads_last_cuda_error) */
  STRADS_ERR_NUMERIC = -5,              /* NaN / Inf met by a kernel (from strads_status)      */
  STRADS_ERR_TIMEOUT = -6,              /* a bounded device-side wait expired                  */
  STRADS_ERR_UNSUPPORTED = -7           /* size beyond a documented limit                      */
} strads_status_t;

typedef enum { STRADS_DENSE_COLMAJOR = 0, STRADS_CSC = 1 } strads_layout_t;

/* flags */
#define STRADS_FLAG_NONE          0u
#define STRADS_FLAG_UNIFORM_DRAW  1u   /* p(j) uniform instead of delta_j^2 + eta (the random
                                          scheduler the paper compares with, Section 5.1)      */
#define STRADS_FLAG_NO_FILTER     2u   /* skip the rho test: keep the first P candidates       */
#define STRADS_FLAG_SIMT_GRAM     4u   /* dense Gram on the FP32 SIMT kernel instead of the
                                          tensor-core kernels                                  */
#define STRADS_FLAG_GRAM_3XTF32   8u   /* dense Gram always by the 3xTF32 tensor-core kernel
                                          (default: a screen on BF16 roundings of the columns,
                                          then an exact FP64 recheck of every pair whose
                                          correlation it puts within 2^-7 + N 2^-25 of rho, so
                                          that Algorithm 1's rho test is decided exactly;
                                          3xTF32 only if the list of such pairs overflows)     */

#define STRADS_FLAG_FULL_GRAM    16u   /* form the conflict bits of ALL P' candidates before the
                                          walk (default: of a leading window of 1.5 P + 128 first,
                                          of all P' only if the walk runs out of the window)    */

#define STRADS_FLAG_ABS_WEIGHT    32u   /* p(j) ~ |delta_j| + eta, Algorithm 1 as printed ("Draw a set U ..."), instead
                                          of Theorem 1's delta_j^2 + eta                         */
#define STRADS_FLAG_DYNAMIC_DEPS  64u   /* dependencies dropped at run time (Section 1, "Dynamic Block Structures";
                                          SAP step 4): a coefficient that is zero and whose last update left it
                                          there (beta_j = 0, delta_j = 0) is taken to couple with nobody -- it
                                          passes the rho test and blocks no other candidate             */

#define STRADS_FLAG_LOGISTIC     128u   /* logistic loss instead of the squared loss (Section 2.1, remark after Eq. 1):
                                          y_i in {0, 1}, F = sum_i [log(1 + exp(m_i)) - y_i m_i] + lambda ||beta||_1 with
                                          the margin m = X beta.  `resid` then holds y - sigma(m), minus the gradient
                                          with respect to m, which plays the residual's part in every step; the
                                          coordinate step is Shotgun's for this loss (curvature at most n_j / 4):
                                          beta_j' = S(beta_j + 4 x_j^T resid / n_j, 4 lambda / n_j).  The margin is kept
                                          in the workspace (strads_margin); strads_round_host is not available.     */

/* limits */
#define STRADS_MAX_CANDIDATES 16384     /* P' <= 16384 (positions in the candidate list are packed into 16 bits
                                           in the lists of pairs; the walk holds P' / 32 mask words per CTA) */
#define STRADS_MAX_C_INIT 1e18f         /* c_init^2 + eta must stay finite in binary32 */
#define STRADS_MAX_SCHEDULERS 8

typedef struct {
  int32_t  layout;                      /* strads_layout_t                                          */
  int64_t  n_rows, n_cols;              /* N, J;  1 <= N,  1 <= J < 2^31                            */
  int64_t  nnz;                         /* CSC: number of stored entries; dense: ignored            */
  int64_t  ld;                          /* dense: floats between column starts, ld >= N, ld % 4 == 0 */
  const float*   x_values;              /* device, 16-byte aligned. dense: [J][ld]; CSC: [nnz]      */
  const int32_t* x_row_idx;             /* device, CSC: [nnz], strictly ascending inside a column   */
  const int64_t* x_col_ptr;             /* device, CSC: [J+1], col_ptr[0] = 0, col_ptr[J] = nnz     */
  const float*   y;                     /* device [N], 16-byte aligned                              */
  float*   beta;                        /* device [J]; in: beta^(0) (normally 0); out: current beta */
  float*   resid;                       /* device [N], 16-byte aligned; written by init: y - X beta */
  float*   delta;                       /* device [J], 16-byte aligned; written by init: c_init     */
  float    lambda;                      /* > = 0                                                    */
  float    eta;                         /* > 0   (paper: 1e-6 in the experiments)                   */
  float    rho;                         /* > 0   (paper: 0.1)                                       */
  float    c_init;                      /* 0 < C <= STRADS_MAX_C_INIT, Algorithm 1's "very large" C; 1e4 recommended */
  int32_t  n_candidates;                /* P': 1 <= P' <= min(J, STRADS_MAX_CANDIDATES)             */
  int32_t  n_keep;                      /* P : 1 <= P <= P'                                         */
  uint64_t seed;                        /* Philox key                                               */
  void*    workspace;                   /* device, 256-byte aligned, strads_workspace_bytes() long  */
  size_t   workspace_bytes;
  void*    stream;                      /* cudaStream_t (NULL = legacy default stream)              */
  uint32_t flags;
  int32_t  n_schedulers;                /* S: scheduler threads taking turns (Section 3); 0 or 1 = one;
                                           1 <= S <= STRADS_MAX_SCHEDULERS and P' <= floor(J / S)       */
} strads_lasso_config_t;

/* Optional per-round outputs; every pointer is a DEVICE address or NULL (= not wanted). */
typedef struct {
  int32_t* cand;      /* [P'] candidates, best first (SAP step 1)                         */
  int32_t* kept;      /* [P]  coefficients that passed the rho test, in walk order; -1 after n_kept */
  float*   dbeta;     /* [P]  signed change beta_j^(t_j) - beta_j^(t_j - 1) per kept entry; 0 after n_kept */
  int32_t* counts;    /* [4]  n_candidates, n_examined, n_kept, n_nonzero_changes          */
  float*   gram;      /* [P'*P'] x_a^T x_b of all candidate pairs in candidate order (debug aid:
                         costs 4 P'^2 bytes of traffic per round; dense X then takes the FP32
                         SIMT Gram kernel, which is the one that can export its values)      */
} strads_round_out_t;

/* Bytes of device workspace that `cfg` needs (pointer fields of cfg are not read). */
int strads_workspace_bytes(const strads_lasso_config_t* cfg, size_t* out_bytes);

/* Algorithm 1's initialisation: n_j = ||x_j||^2 for all j, resid = y - X beta, delta_j = C,
 * round index t = 0.  Validates cfg, creates the handle.  Asynchronous. */
int strads_lasso_init(const strads_lasso_config_t* cfg, strads_handle_t* out_handle);

/* One whole round of Algorithm 1's loop body (SAP steps 1, 2, 4; step 3 is "block size one"
 * for the Lasso, Section 2.1):
 *   1. draw P' candidates without replacement with p(j) ~ delta_j^2 + eta
 *      (Philox4x32-10 word of (seed, t, j); exponential race; best first);
 *   2. walk them best first and keep a candidate when its |correlation| with every candidate
 *      kept before is < rho; stop at P kept;
 *   3. for all kept j, from the same pre-round residual r:
 *        g_j = x_j^T r,  beta_j' = S(beta_j + g_j / n_j, lambda / n_j)     (Eq. 2)
 *      then beta_j <- beta_j', delta_j <- |beta_j' - beta_j|, r <- r - sum_j x_j (beta_j' - beta_j);
 *   4. t <- t + 1.
 * `out` may be NULL.  Asynchronous. */
int strads_round(strads_handle_t h, const strads_round_out_t* out);

/* n_rounds rounds back to back with no host synchronisation in between.
 *
 * Scheduler threads (Section 3, "Implementation Overview" and "Properties"): with n_schedulers = S > 1
 * the coefficients are split into S fixed disjoint sets, scheduler s owning { j : j mod S == s } (the
 * paper assigns them at random; permute the columns for that).  Round t is dispatched by scheduler
 * t mod S, which draws its P' candidates from its own coefficients only (its own p_s(j); the Philox word
 * of (seed, t, j) as before) and filters them; the update of step 3 is unchanged.  delta_j of scheduler s
 * changes only in its own rounds, so its block for round t is fully determined once round t - S is over:
 * strads_run prepares the blocks of up to S - 1 later rounds (steps 1 and 2, on streams of its own) while
 * the update of the current round runs, which is the paper's "each thread has S-fold more time" and gives
 * results identical to running the same rounds strictly one after another (strads_round does that).
 * Each scheduler has its own slice of the workspace.  On return every piece of work has been enqueued and
 * the configured stream waits for all of it.
 *
 * One scheduler, dense X, n_keep <= 4096: the candidates of round t + 1 (Algorithm 1's draw) depend on
 * round t only through the at most P priorities its update changes, so strads_run draws the P' + P best of
 * round t + 1 during round t, on a stream of its own beside the Gram and the walk, from the priorities of
 * round t's start, and round t + 1 starts from that list corrected for the coefficients round t updated
 * (they are struck and entered again with their new keys; the P' smallest remain).  The candidates are
 * exactly those of a draw made at the round's start; the state after strads_run equals that of the same
 * rounds run with strads_round, bit for bit.  Eight rounds are replayed per captured launch sequence, and what is
 * left over of a run as sequences of four, two and one round (with any layout and number of schedulers the rounds
 * of a run are replayed from captured sequences; with several schedulers 16 turns of each per sequence); the
 * streams and events this needs belong to the handle (no device memory is allocated). */
int strads_run(strads_handle_t h, int64_t n_rounds);

/* The same round as strads_round for callers whose state lives in HOST memory: copies
 * beta[J], resid[N], delta[J] host->device, runs one round, copies them back together with
 * the optional host outputs (kept [P], dbeta [P], counts [4]; NULL = not wanted), and waits
 * for the stream.  Host buffers should be pinned for the copies to be asynchronous. */
int strads_round_host(strads_handle_t h, float* beta_host, float* resid_host, float* delta_host,
                      int32_t* kept_host, float* dbeta_host, int32_t* counts_host);

/* Eq. 1 with squared loss from the maintained residual: F = 1/2 ||r||^2 + lambda ||beta||_1,
 * accumulated in FP64.  Synchronises the stream. */
int strads_objective(strads_handle_t h, double* host_out);

/* Split-phase entry points (each is one step of the round, for step-by-step checking).
 * strads_sample : SAP step 1 for the current (delta, seed, t); cand_dev [P'] device.
 * strads_filter : SAP step 2 on a caller-supplied ordered candidate list (device, n_cand <= P');
 *                 kept_dev [P] device, counts_dev [4] device (as strads_round_out_t.counts).
 * strads_update : Eq. 2 + residual + delta refresh for a caller-supplied kept list (device; may be NULL when n_kept is 0;
 *                 distinct indices, n_kept <= P); dbeta_dev [P] device or NULL.
 * None of them advances the round index.  With S > 1 schedulers they act for the scheduler whose turn
 * it is (round index mod S): strads_sample draws from its coefficients, and all three use its slice
 * of the workspace. */
int strads_sample(strads_handle_t h, int32_t* cand_dev);
int strads_filter(strads_handle_t h, const int32_t* cand_dev, int32_t n_cand,
                  int32_t* kept_dev, int32_t* counts_dev, float* gram_dev_or_null);
int strads_update(strads_handle_t h, const int32_t* kept_dev, int32_t n_kept, float* dbeta_dev);

/* Round index t (0-based; the Philox counter).  With beta, resid, delta and the seed it is the
 * whole resumable state.  strads_run keeps the candidates it has drawn ahead for the next round; whoever
 * writes beta, resid or delta directly (a restored checkpoint, priorities set by hand) must call
 * strads_set_round afterwards -- with the current index if it is unchanged -- which discards that list, so
 * that the next round draws from the state as it now is. */
int strads_get_round(strads_handle_t h, int64_t* t_host_out);
int strads_set_round(strads_handle_t h, int64_t t);

/* Cumulative counters since init: totals[0] rounds, [1] candidates examined, [2] coefficients
 * updated (sum of n_kept), [3] non-zero changes.  Synchronises the stream. */
int strads_totals(strads_handle_t h, int64_t* totals_host_out /* [4] */);

/* Reads the device status word (synchronises).  *bits_host_out receives the raw bits;
 * the return value is STRADS_OK, STRADS_ERR_NUMERIC or STRADS_ERR_TIMEOUT. */
#define STRADS_STATUS_SAMPLER_REFINED 1u   /* informational: the sampler needed extra select passes */
#define STRADS_STATUS_NONFINITE       2u   /* a gradient x_j^T r was NaN or Inf                     */
#define STRADS_STATUS_WAIT_EXPIRED    4u   /* a bounded wait in a kernel gave up                     */
#define STRADS_STATUS_GRAM_FALLBACK   8u   /* informational: the dense Gram's BF16 screen left more
                                              borderline pairs than its list holds; 3xTF32 was used  */
int strads_status(strads_handle_t h, uint32_t* bits_host_out);

/* The error contract of the bounded waits ("nothing waits without a bound").  Every device-side wait of the
 * round -- the mbarrier waits of the dense Gram's TMA / tensor-core pipeline (SAP step 2) and the grid-wide
 * barrier of the CSC on-demand walk -- counts its iterations; past the limit the CTA raises
 * STRADS_STATUS_WAIT_EXPIRED, stops issuing work, releases its tensor memory and returns, so the launch ends and
 * strads_status reports STRADS_ERR_TIMEOUT.  From then on the round's outputs and beta / resid / delta are
 * undefined, and the CSC walk does nothing on this handle, until strads_recover has been called:
 *   restore beta, resid, delta from a copy of your own, strads_recover, strads_set_round, carry on.
 * strads_set_wait_limit: iteration limit for all those waits on this handle (0 = the kernels' defaults, which
 *   amount to seconds); synchronises the stream and drops the captured launch sequence of strads_run.
 * strads_inject_stall: makes a wait of the NEXT launches run out, so that the path above can be exercised: with
 *   STRADS_STALL_WALK_BARRIER the arrival counter of the CSC walk's barrier is set to a value no barrier completes
 *   from; with STRADS_STALL_GRAM_LOADS the dense Gram's producer withholds its operand loads (until
 *   strads_recover).  Nothing faults or hangs: the waits give up.  Refused (STRADS_ERR_INVALID_ARG) unless a
 *   limit of at most STRADS_STALL_MAX_WAIT_LIMIT iterations is in force, so that giving up takes milliseconds.
 * strads_recover: waits for the stream, clears the status word and the barrier state, ends an injected stall. */
#define STRADS_STALL_WALK_BARRIER 1
#define STRADS_STALL_GRAM_LOADS   2
#define STRADS_STALL_MAX_WAIT_LIMIT 65536u
int strads_set_wait_limit(strads_handle_t h, uint32_t iterations);
int strads_inject_stall(strads_handle_t h, int32_t which);
int strads_recover(strads_handle_t h);

/* STRADS_FLAG_LOGISTIC: the margin m = X beta, FP32, device [N] (points into the workspace); with beta, resid,
 * delta and the round index it is the resumable state.  STRADS_ERR_INVALID_ARG without the flag. */
int strads_margin(strads_handle_t h, float** dev_ptr_out);

/* ||x_j||^2 as computed by init, FP64, device [J] (points into the workspace). */
int strads_colnorm2(strads_handle_t h, const double** dev_ptr_out);

/* Optional step timing with CUDA events on the handle's stream (n_schedulers == 1 only: with more, the
 * steps of different rounds overlap and have no separate times).  After strads_profile_begin the next
 * max_rounds rounds (strads_round / strads_run / strads_round_host; strads_run then launches kernel by kernel
 * instead of replaying its graph) record an event at every step boundary; strads_profile_end waits for the
 * stream and returns the summed device time in milliseconds over *rounds rounds of
 *   ms[0] candidate sampling,
 *   ms[1] packing the candidate columns (dense tensor-core path; 0 otherwise),
 *   ms[2] the Gram kernels (of the candidate window, or of all candidates when no window is used),
 *   ms[3] the greedy walk, plus the whole-list retry when the window was too short,
 *   ms[4] the update.
 * Events are host-side driver objects; no device memory is allocated. */
int strads_profile_begin(strads_handle_t h, int64_t max_rounds);
int strads_profile_end(strads_handle_t h, double* ms_host_out /* [5] */, int64_t* rounds_host_out);

int strads_destroy(strads_handle_t h);

/* (No counterpart in the paper: a packaging variant of SAP step 1.)
 * The candidate draw of strads_sample for callers that must not allocate device memory -- code that
 * runs inside another component's memory pool, plugins whose host forbids cudaMalloc after start-up,
 * latency-critical loops.  It needs no handle and no workspace: the scratch memory of the select
 * passes lives in a fixed array inside the library (about 65 KB on every GPU that loads it, until the
 * process exits), which limits it to n_candidates <= STRADS_STATIC_MAX_CANDIDATES; larger requests
 * return STRADS_ERR_UNSUPPORTED.  The call allocates nothing (no cudaMalloc / cudaFree, no allocating
 * library routine).
 *   delta_dev [n_cols] device, 16-byte aligned; cand_dev [n_candidates] device: the same ordered list
 *   strads_sample gives for the same (delta, eta, seed, t, flags); stream: cudaStream_t.
 * Asynchronous on `stream`.  The first call on a device looks up the array's device address (with
 * that device current); make that first call before any stream capture begins.  All calls on one
 * device share the array and it keeps the previous call's contents (the call clears what must start
 * at zero), so two calls that overlap on the GPU -- different streams, or different threads -- race:
 * serialise them. */
#define STRADS_STATIC_MAX_CANDIDATES 4096
int strads_sample_static(const float* delta_dev, int64_t n_cols, float eta, uint64_t seed, uint64_t t,
                         int32_t n_candidates, uint32_t flags, int32_t* cand_dev, void* stream);

const char* strads_error_string(int code);
/* Text of the last CUDA error seen by this library on the calling thread ("" if none). */
const char* strads_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* STRADS_H_ */
