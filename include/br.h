/*
 * BalanceRoute routing step for data-parallel LLM decode, C ABI.
 *
 * One *routing instance* is a fleet of G decode workers with B request slots
 * each plus a waiting set of prefill-completed requests (the cluster snapshot of
 * Section 5, Eq. "cluster-snapshot").  br_step advances a batch of independent
 * instances by one decode step k:
 *
 *   ARRIVE   new requests join R_wait(k) in arrival order      (Section 2.2)
 *   PREDICT  c_hat maintenance and horizon projection (H > 0)   (Eqs. 3-6, Appendix "Refresh logic")
 *   ROUTE    two-stage admission by F-score                     (Eq. 1 / Eq. 2, Algorithms 1 and 2)
 *   RECORD   per-worker loads L_g(k) and (max, min, sum)        (Section 3.1, Section 5.1 "Metrics")
 *   ADVANCE  every running request ends or grows by one token   (Section 2.2)
 *
 * All array arguments are DEVICE pointers owned by the caller unless a comment
 * says "host".  The library keeps no pointer beyond a call, except those baked
 * into a captured graph (br_graph_capture), which must stay valid until
 * br_destroy.  Calls are asynchronous on the stream given in the batch and
 * return a host status at once; nothing aborts, traps or prints.  A br_ctx must
 * not be used from two host threads at the same time.
 */
#ifndef BR_H_
#define BR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BR_VERSION 102

/* status codes returned by every entry point */
#define BR_OK        0
#define BR_EINVAL   -1   /* null / misaligned pointer, or a size outside the limits below */
#define BR_ERANGE   -2   /* a value range that the integer packing cannot represent       */
#define BR_ECUDA    -3   /* a CUDA runtime call failed; br_strerror gives its text        */
#define BR_ENOMEM   -4   /* host or device allocation failed (br_create, host-buffer path)*/
#define BR_ESTATE   -5   /* call order violated (e.g. br_graph_step before capture)       */
#define BR_ELIMIT   -6   /* br_step_host_static: the batch does not fit BR_STATIC_STAGE_BYTES */

/* compiled limits */
#define BR_MAX_G      64
#define BR_MAX_H      80     /* the lookahead the paper deploys (Section 5.1 "Our methods")   */
#define BR_MAX_B     256     /* B must be a multiple of 8                     */
#define BR_MAX_W    4096     /* W must be a multiple of 4                     */
#define BR_MAX_RMAX   16     /* Stage-2 window; beyond 5 entries the subsets are searched by
                                meeting in the middle, which needs G >= 2 (Eq. 1) or Eq. 2
                                parameters without a flat segment and H <= 16       */

#define BR_EMPTY_SLOT INT32_MIN  /* act_base value of a free slot              */

/* per-instance status bits written to br_load_out.status */
#define BR_ST_QUEUE_OVERFLOW  1u  /* at least one arrival was dropped (queue at W)   */
#define BR_ST_ITER_CAP        2u  /* a routing loop hit its hard iteration bound     */
#define BR_ST_BAD_STATE       4u  /* nact/occ/queue length inconsistent with limits  */

typedef struct br_ctx br_ctx;

/*
 * Parameters, host memory, copied by br_create.  "default" = value used when the
 * field is negative (or zero where zero is not meaningful).
 */
typedef struct {
    int32_t B;              /* slots per worker (max concurrency B, Section 2.2)             */
    int32_t W;              /* capacity of the waiting queue                                  */
    int32_t R_max;          /* Stage-2 window (Algorithm 1); <= 0 -> 4; at most BR_MAX_RMAX  */
    int32_t S_greedy;       /* Stage-1 / Stage-2 threshold on total free slots; < 0 -> 2 G   */
    double  alpha, beta, gamma; /* Eq. 2 parameters; ignored when score_mode == 0            */
    int32_t delta_T;        /* c_hat refresh period; <= 0 -> max(1, H / 2)                   */
    float   gate;           /* confidence gate on p_fin; < 0 -> 0.5                          */
    float   c_floor;        /* lower bound of c_hat; < 0 -> 1                                */
    int32_t score_mode;     /* 0: Eq. 1 in integers (needs H == 0); 1: Eq. 2 in fp64; < 0 -> 0 if H == 0 else 1 */
    int32_t term_mode;      /* 0: requests never end; 1: every slot ends with the same probability p per
                               step, independently (term_cdf); 2: end when a 24-bit Philox uniform <
                               term_probs[slot][0]; 3: every request carries its output length o_i
                               (Section 2.2): admitted at step x it runs at steps x .. x + o_i - 1
                               (act_end, waiting_queue.o, out_tab)                              */
    const uint32_t *term_cdf; /* device [B], term_mode 1: term_cdf[j] = floor(2^32 (1 - (1-p)^(j+1))), the
                               CDF of the number of slots skipped before the next ending one.  Per
                               worker and step the ending slots are walked by these gaps: draw t is
                               word t % 4 of the Philox block (k, g, TERM, t / 4), gap = #{j : u >= term_cdf[j]} */
    const uint32_t *arr_cdf;/* device [rows][arr_len] Poisson CDF thresholds; the row for instance i
                               at step k is i * arr_inst_stride + k % arr_period; NULL -> no arrivals */
    int32_t arr_len, arr_period, arr_inst_stride;
    const int32_t *len_tab; /* device [2^len_tab_log2] inverse-CDF table of prompt lengths   */
    int32_t len_tab_log2;
    int32_t burst_every, burst_size; /* burst_size extra arrivals when k > 0 and k % burst_every == 0 */
    int32_t s_max;          /* largest prompt length the caller will ever enqueue (range proof) */
    int32_t threads;        /* threads per instance (multiple of 32, <= 256); <= 0 -> chosen from G*B, H and the batch size */
    int32_t inst_per_block; /* instances per thread block when an instance runs on one warp (1..8); <= 0 -> 4 */
    int32_t pred_mode;      /* H > 0 only.  0: c_hat from the classifier output term_probs (Eqs. 3-5 and the
                               refresh rules); 1: c_hat = min(r_i(k), H) from the known lifetimes, the
                               perfect-lookahead reference of Section 5.1 "Our methods" (needs term_mode 3;
                               term_probs, act_chat0 and act_kref are not used and may be NULL)        */
    const int32_t *out_tab; /* device [2^out_tab_log2] inverse-CDF table of output lengths o_i >= 1 given to
                               arrivals in term_mode 3: word j % 4 of the Philox block (k, j / 4, 3, 0) */
    int32_t out_tab_log2;
} br_params;

/* running requests; instance i occupies row first_instance + i of every array */
typedef struct {
    int64_t  *load;       /* [N][G]   L_g at the start of the step (sum of cur over the worker)  */
    int32_t  *nact;       /* [N][G]   |A_g|                                                     */
    uint64_t *occ;        /* [N][G][ceil(B/64)] bit b set <=> slot b is occupied                */
    int32_t  *act_base;   /* [N][G][B] cur - k of the request in the slot (constant while it
                                       runs: cur = s_i + (k - x_i)), BR_EMPTY_SLOT if free      */
    uint32_t *act_id;     /* [N][G][B] request id per slot; may be NULL                         */
    float    *act_chat0;  /* [N][G][B] c_hat at the last refresh (H > 0 only, else may be NULL) */
    uint8_t  *act_kref;   /* [N][G][B] step of the last refresh modulo 256 (H > 0 only)         */
    int32_t  *act_end;    /* [N][G][B] term_mode 3: the step at whose end the request finishes
                                       (x_i + o_i - 1); else may be NULL                         */
    int32_t  *step;       /* [N]      decode step k                                             */
    uint64_t *seed;       /* [N]      Philox key of the instance                                */
    uint32_t *next_id;    /* [N]      id given to the next arrival                              */
} br_worker_state;

/* waiting requests in arrival order; entries [n, W) are ignored */
typedef struct {
    int32_t  *s;          /* [N][W] prompt length s_i = w_i^(1)                                 */
    uint32_t *id;         /* [N][W] request id                                                  */
    int32_t  *n;          /* [N]    current length                                              */
    int32_t  *o;          /* [N][W] term_mode 3: output length o_i of the waiting request (latent to
                                    the router, carried along for the simulation); else may be NULL */
} br_waiting_queue;

typedef struct {
    int32_t n_instances;    /* instances in this call                                           */
    int32_t first_instance; /* row offset into every per-instance array, state and outputs alike   */
    int32_t n_steps;        /* consecutive decode steps run by this one launch; <= 0 -> 1.  With
                               n_steps > 1, term_probs, assign_out and every br_load_out array
                               hold n_steps consecutive per-step blocks of n_instances rows,
                               indexed from row 0 (first_instance must then be 0)              */
    void   *stream;         /* cudaStream_t                                                     */
} br_instance_batch;

typedef struct {
    int64_t  *load;       /* [N][G]  L_g(k) after this step's admissions                        */
    int64_t  *trace;      /* [N][3]  (max_g L_g, min_g L_g, sum_g L_g); gives max-min, I(k), max/mean */
    int32_t  *status;     /* [N]     BR_ST_* bits; may be NULL                                  */
    uint32_t *counters;   /* [N][4]  this step: dropped arrivals, admissions, Stage-1 iterations,
                                     Stage-2 pops; may be NULL                                  */
    double   *fscore;     /* [N][W][G] optional: F_g({i}) of every waiting request before the
                                     first admission (0 beyond the queue length); NULL in timed runs */
    uint32_t *phase_cycles; /* [N][8] optional: SM clock cycles this step spent in ARRIVE, PREDICT,
                                     Stage 1, Stage 2, RECORD + queue compaction, ADVANCE (the split the
                                     paper reports for its dispatcher: preparation / Stage 1 / Stage 2),
                                     then the launch's state-load prologue and its total from kernel
                                     entry to the state write-back; may be NULL */
} br_load_out;

/*
 * Creates a context for fleets of G workers and lookahead H (H = 0: BR-0).
 * Validates sizes against the limits above and proves that queue keys, loads and
 * Eq. 1 scores fit the 32-bit arithmetic used on the device (else BR_ERANGE):
 * s_max * 2^ceil(log2 W) < 2^31, B * (s_max + 2^22) < 2^31 (a request may run for at
 * most 2^22 steps), G * R_max * s_max < 2^31.  Prompt lengths must be >= 1.
 * Allocates only a small host object.  *out is set on BR_OK only.
 */
int br_create(int32_t G, int32_t H, const br_params *params, br_ctx **out);

/*
 * One decode step (or batch.n_steps of them) for batch.n_instances instances.
 * Mutates worker_state and waiting_queue in place.
 *   term_probs  [N][G][B][H] fp32 termination-classifier output for this step: entry h-1 is
 *               the probability that the request ends at in-window step h given that it is
 *               still running; NULL allowed when H == 0 and term_mode != 2
 *   assign_out  [N][W] per queue position (as of after ARRIVE): g * B + slot of the admission,
 *               -1 if the request keeps waiting or the position is beyond the queue
 * Returns BR_EINVAL for null or misaligned (16-byte) array pointers and n_instances < 0,
 * BR_ECUDA if the launch failed.  n_instances == 0 is a no-op returning BR_OK.
 */
int br_step(br_ctx *ctx, const br_instance_batch *batch, br_worker_state *worker_state,
            br_waiting_queue *waiting_queue, const float *term_probs, int32_t *assign_out,
            br_load_out *load_out);

/*
 * Latency path: records one br_step launch with these arguments into a CUDA graph
 * owned by ctx (replacing an earlier one); br_graph_step replays it on the stream
 * given at capture.  The step counter lives in worker_state.step, so every replay
 * advances by batch.n_steps steps; the caller refreshes term_probs in place.
 */
int br_graph_capture(br_ctx *ctx, const br_instance_batch *batch, br_worker_state *worker_state,
                     br_waiting_queue *waiting_queue, const float *term_probs,
                     int32_t *assign_out, br_load_out *load_out);
int br_graph_step(br_ctx *ctx);

/*
 * Host-buffer variant: every array pointer in worker_state, waiting_queue, term_probs,
 * assign_out and load_out is a HOST pointer (pinned memory gives asynchronous copies).
 * Copies the snapshot to device staging owned by ctx (grown on demand with cudaMalloc),
 * runs the step, copies state and results back and synchronises the stream.  Batches of 512
 * instances or more go through in chunks of instances on three internal streams (created on
 * first use), so that uploads, kernels and downloads of different chunks overlap.
 * h2d_bytes / d2h_bytes, if not NULL, receive the bytes moved in each direction.
 * batch.n_steps must be 1 and batch.first_instance 0.
 */
int br_step_host(br_ctx *ctx, const br_instance_batch *batch, br_worker_state *worker_state,
                 br_waiting_queue *waiting_queue, const float *term_probs, int32_t *assign_out,
                 br_load_out *load_out, int64_t *h2d_bytes, int64_t *d2h_bytes);

/*
 * br_step_host for callers that must not allocate.  (The paper has no counterpart: this entry
 * point exists for the library's users, not for the method.)
 *
 * Who needs it: code that runs where device allocation is forbidden or unsafe -- inside a
 * latency-critical serving loop whose memory is fully pre-planned, in a process whose CUDA
 * memory pool is owned by another framework and sized to the last byte, or in a callback /
 * signal-like context where cudaMalloc (which may synchronise the device and take driver
 * locks) can stall or deadlock.  br_step_host grows a staging buffer with cudaMalloc on
 * demand; this variant never calls cudaMalloc, cudaFree or any allocating routine.
 *
 * The device-side staging is a fixed array of BR_STATIC_STAGE_BYTES built into the library
 * image, so every GPU that loads the library holds that much memory until the process exits.
 * A batch whose snapshot plus outputs (each array padded to 256 bytes) exceeds it is rejected
 * with BR_ELIMIT before anything is copied; load_out->fscore must be NULL (BR_EINVAL).
 * Otherwise arguments, results and status codes are those of br_step_host.
 *
 * The first call on each device looks up the array's device address (a CUDA runtime query
 * made with that device current; no allocation) and keeps it for later calls.  Make that first
 * call before any stream capture begins on the thread; the entry point itself ends with a stream
 * synchronisation and therefore never belongs inside a capture.  All calls on a device share the
 * one array, which still holds the previous call's data: inputs are overwritten by the copies of
 * this call and the output blocks are cleared first, but two calls that overlap on the GPU
 * (different streams, or different host threads) race on it -- serialise them.  If a CUDA call
 * fails after copies have been queued, the stream is drained before the error is returned.
 */
#define BR_STATIC_STAGE_BYTES (8u << 20)
int br_step_host_static(br_ctx *ctx, const br_instance_batch *batch, br_worker_state *worker_state,
                        br_waiting_queue *waiting_queue, const float *term_probs,
                        int32_t *assign_out, br_load_out *load_out, int64_t *h2d_bytes,
                        int64_t *d2h_bytes);

/*
 * F-score matrix alone (Eq. 1 / Eq. 2 for single requests): for n_requests prompt lengths s
 * and per-instance projected loads Lh [N][G][H+1] (offset 0 = L_g(k)), writes
 * F [N][n_requests][G] in fp64 and, if best_g is not NULL, argmax_g per request
 * (lowest g on ties) restricted to workers with cap[g] > 0 (cap [N][G], may be NULL).
 * This is the pool-bypass scorer of Appendix "Pool-bypass deployment path for BR-0"
 * when H = 0 and Lh holds virtual loads.
 */
int br_fscore(br_ctx *ctx, const br_instance_batch *batch, const int32_t *s, int32_t n_requests,
              const int64_t *Lh, const int32_t *cap, double *F, int32_t *best_g);

/*
 * The Stage-2 subproblem alone, solved exactly on windows of up to 32 requests (Algorithms 1 and 2,
 * Stage 2; Appendix "Bit-set subset selection": the score depends on Q only through Delta(Q)).
 * For each of batch.n_instances problems: win [N][R] holds the prompt lengths of the window
 * (1 <= R <= 32; bit j of a mask selects entry j), margins [N][H+1] the worker's m_{g,h} (H = 0:
 * m_g), lim [N] the largest subset size (the worker's free slots).  Writes best_mask [N] = the
 * non-empty subset with |Q| <= lim and the highest F_g(Q) (Eq. 1 / Eq. 2 as in br_step), lowest mask
 * on ties, 0 if lim < 1; best_F [N] (may be NULL) its score.  Up to 12 requests all 2^R - 1 subsets
 * are enumerated; from 13 on the window is split in two halves that meet in the middle: the best
 * subset has the largest reachable Delta at or below the score's peak or the smallest above it (the
 * appendix's two-probe rule), found by binary searches over the sorted subset sums of one half, per
 * subset size.  That rule needs a score that is strictly monotone on both sides of its peak: Eq. 1
 * with G >= 2, or Eq. 2 with H <= 16 and no segment slope within rounding distance of zero (checked
 * by br_create); otherwise windows of up to 20 requests are enumerated and larger ones refused.
 * Device pointers; asynchronous on batch.stream; BR_EINVAL for null pointers, R outside [1, 32], or
 * R > 20 without the two-probe rule.
 */
int br_best_subset(br_ctx *ctx, const br_instance_batch *batch, const int32_t *win, int32_t R,
                   const int64_t *margins, const int32_t *lim, uint32_t *best_mask, double *best_F);

/*
 * Pool-bypass dispatch for BR-0 (Appendix "Pool-bypass deployment path for BR-0"; ctx must have
 * H = 0, else BR_EINVAL).  For each instance the n_requests prompt lengths s [N][n_requests] are
 * routed one at a time in arrival order: request i goes to argmax_g F_g(s_i) (Eq. 1 with the
 * context's coefficients, lowest g on ties) over the workers with inflight[g] < inflight_cap[g],
 * where the margins m_g = M - L_g come from the virtual loads virtual_load [N][G] (running plus
 * requests that were dispatched and have not started yet).  The chosen worker's virtual load grows by s_i and its
 * inflight count by one before the next request is scored.  worker_out [N][n_requests] receives
 * the worker, -1 when every worker is at its cap; virtual_load and inflight are updated in place.
 * Device pointers, asynchronous on batch.stream.
 */
int br_bypass_dispatch(br_ctx *ctx, const br_instance_batch *batch, const int32_t *s, int32_t n_requests,
                       int64_t *virtual_load, int32_t *inflight, const int32_t *inflight_cap,
                       int32_t *worker_out);

/*
 * Empirical-survival estimator of c_hat (Appendix "Estimator realizations", "Empirical-survival";
 * Eqs. 3-5), for contexts with H >= 1.  hist_sorted [n_hist] holds recorded output lengths in
 * ascending order, hist_prefix [n_hist + 1] their prefix sums (hist_prefix[j] = sum of the first
 * j entries).  For each of count requests with age[i] tokens produced so far:
 *   p_fin = #{age < o <= age + H} / #{o > age},  mu_rem = mean of (o - age) over that window,
 *   c_hat = (1 - p_fin) H + p_fin mu_rem clipped to [0, H]   (fp64, stored as fp32);
 * with no recorded output inside the window p_fin = 0, mu_rem = H and c_hat = H.  p_fin and
 * mu_rem [count] may be NULL.  Device pointers; asynchronous on stream (a cudaStream_t).
 * BR_EINVAL for null pointers, H = 0, n_hist < 1 or count < 0.
 */
int br_survival_chat(br_ctx *ctx, void *stream, const int32_t *hist_sorted, const int64_t *hist_prefix,
                     int32_t n_hist, const int32_t *age, int64_t count, float *c_hat, double *p_fin,
                     double *mu_rem);

/*
 * Range-checked build (libbr_dbg.so, compiled with -DBR_BOUNDS; the paper has no counterpart).  In
 * that build every per-instance array of the step kernels -- shared memory and global rows -- is
 * indexed through a span that knows its length: an index outside it is counted and redirected to a
 * sink, so nothing outside the array is read or written and the kernel ends normally.
 * br_debug_bounds_hits synchronises the device and returns the count since the library was loaded;
 * br_debug_bounds_selftest indexes a span over the four device ints it is given three times out of
 * range (into the sink) and returns how many hits that added (3).  Both return -1 in the normal
 * build, BR_ECUDA if a CUDA call fails.
 */
int br_debug_bounds_hits(void);
int br_debug_bounds_selftest(int32_t *four_ints);

/* Frees the context, its staging buffers and graph.  NULL is accepted. */
int br_destroy(br_ctx *ctx);

/* Text for a status code; for BR_ECUDA the text of the last CUDA error seen by this library. */
const char *br_strerror(int status);
int br_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BR_H_ */
