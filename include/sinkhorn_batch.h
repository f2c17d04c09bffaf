/*
 * sinkhorn_batch.h — C ABI of the shrinking-active-set batched log-domain
 * Sinkhorn library for NVIDIA B200 (sm_100a).
 *
 * W independent entropic optimal-transport problems ("lanes") are solved side by
 * side.  Problem statement (paper Eq. 1): positive unit-mass marginals
 * a in R^n, b in R^m, cost C_ij = |x_i - y_j|^2 recomputed from the point clouds,
 * regularisation eps.  One cycle is the pair of scaling updates of Eq. 3 in log
 * form,
 *      f_i <- eps (log a_i - LSE_j((g_j - C_ij)/eps)),
 *      g_j <- eps (log b_j - LSE_i((f_i - C_ij)/eps)),
 * and the plan is pi_ij = exp((f_i + g_j - C_ij)/eps); it is never stored.
 * After each audited cycle a lane's row residual is screened, screen-positive
 * lanes get the two-sided check of Eq. 5, and lanes that pass are retired at
 * completion depth l_t (Section "Screen, verify, and compact").  What happens to
 * a retired lane is the execution mode (Section "Execution modes and fallback").
 *
 * Conventions
 *   - Every data pointer is DEVICE memory owned by the caller unless it says
 *     "host".  Inputs are const and never modified.  The library allocates no
 *     device memory: all of its state lives in the caller's workspace.  (Host side, a
 *     handle borrows a 128-byte pinned block and two events from a small per-device pool
 *     that the library keeps for the life of the process.)
 *   - All work is enqueued on the stream given at creation.
 *   - Every call returns an skb_status; nothing throws or aborts.  The text of
 *     the last error is available from sinkhorn_batch_last_error().
 *   - There is no CPU path: every step runs in CUDA kernels.
 */
#ifndef SINKHORN_BATCH_H
#define SINKHORN_BATCH_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct skb_batch skb_batch; /* opaque host object */

typedef enum {
    SKB_OK = 0,
    SKB_ERR_NULL = 1,      /* a required pointer is null */
    SKB_ERR_SHAPE = 2,     /* W, n, m, d < 1 or an unsupported combination */
    SKB_ERR_VALUE = 3,     /* tol <= 0, max_iter < 1, bad enum, non-finite or non-positive input */
    SKB_ERR_WORKSPACE = 4, /* workspace missing, misaligned (256 B) or too small */
    SKB_ERR_STATE = 5,     /* call not valid in the batch's current state */
    SKB_ERR_CUDA = 6       /* a CUDA call or a kernel reported an error */
} skb_status;

/* What is done with a lane that passed the two-sided check. */
typedef enum {
    SKB_ACTIVE = 0, /* retire and physically compact: later kernels run at survivor width A_k */
    SKB_MASKED = 1, /* freeze its potentials, keep it in place: kernels stay at width W        */
    SKB_STATIC = 2, /* keep updating every lane until the deepest lane passes (l_max)          */
    SKB_MASKED_EXIT = 3 /* as MASKED, but the thread blocks of a frozen lane return at once: a     */
                        /* launch slot per lane, no pair work.  NOT the paper's logical-mask       */
                        /* control (which keeps W * l_max slots of work, Section "controls"); an   */
                        /* extra arm that asks whether physically moving survivors still pays on a  */
                        /* kernel that can skip lanes.  Results are bit-identical to MASKED.        */
} skb_mode;

typedef enum { SKB_F32 = 0, SKB_BF16 = 1 } skb_dtype;           /* storage type of x and y only */
/* Arithmetic of the pair terms log2 pi_ij and their exponentials. */
typedef enum {
    SKB_COMPUTE_AUTO = 0,  /* F32 (TENSOR where eligible), or MIXED when some lane's cost/eps  */
                           /* range is beyond fp32 for the tolerance asked for: scaled squared */
                           /* radius log2(e)/eps * max|x - centre|^2 above 512 * min(1, tol/1e-3) */
    SKB_COMPUTE_F32 = 1,   /* fp32 exponents and exponentials                                  */
    SKB_COMPUTE_MIXED = 2, /* float64 exponents (half-rate FP64 pipe), fp32 exponentials       */
    SKB_COMPUTE_F64 = 3,   /* float64 throughout, software exp2: the slow validation arithmetic */
    SKB_COMPUTE_TENSOR = 4 /* bf16 x, y only, d a multiple of 64 up to 512: cross term on the   */
                           /* tensor cores (fp32 accumulate), fp32 exponentials; what AUTO     */
                           /* picks for such inputs                                            */
} skb_compute;

typedef enum {
    SKB_LANE_RUNNING = 0,
    SKB_LANE_DONE = 1,       /* passed the two-sided check at its depth                    */
    SKB_LANE_ITER_LIMIT = 2, /* did not pass within max_iter cycles; depth = max_iter      */
    SKB_LANE_NONFINITE = 3   /* a potential or residual became non-finite; output invalid  */
} skb_lane_status;

typedef struct {
    int W, n, m, d;        /* lanes, source points, target points, dimension               */
    int xy_dtype;          /* skb_dtype                                                    */
    int mode;              /* skb_mode                                                     */
    int compute;           /* skb_compute                                                  */
    int max_iter;          /* cycle cap per lane, >= 1                                     */
    int audit_every;       /* audit after every k-th cycle, >= 1                           */
    float tol_screen;      /* row-screen threshold; <= 0 means "same as tol"               */
    int column_split;      /* 0 = automatic; 1, 4 or 32 forces how many lanes of a warp     */
                           /* share one row's columns in the update kernel (tuning knob)  */
    int cost_form;         /* 0 = chosen per lane from its scaled radius; 1 = expanded     */
                           /* |x|^2+|y|^2-2x.y everywhere; 2 = difference |x-y|^2 everywhere */
    void *stream;          /* cudaStream_t (0 = legacy default stream)                     */
    void *workspace;       /* device, 256-byte aligned                                     */
    size_t workspace_bytes;
    float guard_band;      /* guard band around the thresholds with float64 escalation     */
                           /* (Section 5, stress test of near-threshold accept decisions): */
                           /* a lane whose row screen lies within this RELATIVE distance   */
                           /* of tau_screen or tau_stop (at least 1e-7 absolute) has its   */
                           /* row residual re-evaluated from the raw inputs in float64 and */
                           /* is decided by that value.  Negative = off.  0 = default:     */
                           /* 2.5e-4 for d <= 32, off for deeper lanes, where one lane's   */
                           /* re-evaluation is n*m*d float64 multiply-adds in a launch of  */
                           /* its own per cycle and is only done at a width the caller     */
                           /* names (the tensor-core path's own evaluation error is up to  */
                           /* 1 % of tol).  Costs a raw copy of x and y in the workspace   */
    int lane_capacity;     /* lanes the batch can take in over its life: 0 or W = the W of  */
                           /* create only; more (ACTIVE mode) lets sinkhorn_batch_refill    */
                           /* put new problems into the slots finished lanes have freed;    */
                           /* every per-lane output then has lane_capacity entries          */
} skb_config;

/* Bytes of device workspace a batch with this shape, dtype, mode and compute type
 * needs.  Returns 0 if the configuration is invalid. */
size_t sinkhorn_batch_workspace_bytes(const skb_config *cfg);

/*
 * Create a batch (Eq. 1 inputs) and enqueue its set-up kernels.
 *   x   [W, n, d] row-major, fp32 or bf16 per cfg->xy_dtype      (device)
 *   y   [W, m, d]                                                (device)
 *   a   [W, n] fp32, > 0, each lane sums to 1                    (device)
 *   b   [W, m] fp32, > 0, each lane sums to 1                    (device)
 *   eps [W]    fp32, > 0, per-lane regularisation                (device)
 *   tol        two-sided stopping tolerance tau_stop of Eq. 5    (> 0)
 * Potentials start cold, f = g = 0 (sinkhorn_batch_warm_start replaces them).  Inputs are
 * copied into the workspace in the kernels' own layout; they may be freed once the stream
 * has passed this call.  Non-positive weights or eps and non-finite coordinates are
 * detected on the device and reported as SKB_ERR_VALUE by drain, or by a later step once
 * the control block it reads back asynchronously has arrived.
 * The call waits for its set-up kernels (their time is SKB_PHASE_CREATE of
 * sinkhorn_batch_stats); with SKB_COMPUTE_AUTO it first waits for the lanes' cost range to
 * come back from the device, because the choice of arithmetic decides the layout.
 * On success *out holds the handle; the caller releases it with
 * sinkhorn_batch_destroy (the workspace stays the caller's).
 */
skb_status sinkhorn_batch_create(const void *x, const void *y, const float *a, const float *b,
                                 const float *eps, float tol, const skb_config *cfg,
                                 skb_batch **out);

/*
 * Warm proposal (Section "Initialization and repeated couplings"): start from the caller's
 * potentials instead of f = g = 0.
 *   f0 [W, n], g0 [W, m]  float64, device, the paper's convention pi = exp((f + g - C)/eps);
 *                         either may be null (that side stays cold).  Non-finite values are
 *                         reported as SKB_ERR_VALUE like bad inputs.
 *   audit_initial != 0    the proposal itself is audited (row screen, two-sided check of
 *                         Eq. 5) before any update: a lane whose proposal already passes
 *                         retires at depth 0 with the proposal as its output and its
 *                         measured residuals; the others go on from it.
 * Valid only before the first step/drain (SKB_ERR_STATE afterwards).  Enqueues one kernel.
 */
skb_status sinkhorn_batch_warm_start(skb_batch *h, const double *f0, const double *g0, int audit_initial);

/*
 * Replace finished lanes by new problems (the paper's related work on dynamic batching: completed
 * problems are replaced so that the width does not collapse; compaction keeps the survivors in a
 * dense prefix, so the free slots are the ones past the current width).
 *   x [count, n, d], y [count, m, d], a [count, n], b [count, m], eps [count]   as in create (device)
 *   first_lane (host out, may be null): the new problems become lanes first_lane .. first_lane+count-1
 *   in every per-lane output.
 * ACTIVE mode only; needs count free slots (SKB_ERR_STATE otherwise; the call synchronises the stream
 * to learn the width) and count unused lanes of cfg->lane_capacity (SKB_ERR_SHAPE).  The new lanes
 * start cold and run with the arithmetic the batch was created with (SKB_COMPUTE_AUTO chose it from
 * the first lanes' cost range: name the arithmetic where later problems may have a smaller eps or a
 * wider cloud); their depths count their own
 * cycles, max_iter applies to each lane's own count, audits stay on the batch's cycle grid.  The
 * slot identity of Eq. 7 still holds: slots = sum_k A_k = sum of all lanes' depths.
 */
skb_status sinkhorn_batch_refill(skb_batch *h, const void *x, const void *y, const float *a, const float *b,
                                 const float *eps, int count, int *first_lane);

/* Enqueue `cycles` full cycles (both legs of Eq. 3 plus screen, two-sided check and
 * retirement after every audited one).  Never synchronises: each call leaves an asynchronous
 * copy of the device's control block behind and looks, without waiting, whether an earlier
 * one has arrived; from it the launch width follows the survivors and device-side errors
 * (bad input values, a bounded wait that ran out) are returned.  Cycles past the point where
 * every lane is finished are no-ops. */
skb_status sinkhorn_batch_step(skb_batch *h, int cycles);

/* Run until every lane is retired (passed, hit max_iter, or went non-finite), then
 * synchronise the stream.  *cycles_run (host, may be null) receives the number of
 * complete cycles executed, i.e. the largest depth. */
skb_status sinkhorn_batch_drain(skb_batch *h, int *cycles_run);

/* Number of lanes still running (host out).  Synchronises the stream. */
skb_status sinkhorn_batch_active(skb_batch *h, int *n_active);

/* Potentials in the paper's convention pi = exp((f + g - C)/eps), original lane order.
 * f [L, n], g [L, m] device out, either may be null (L = lane_capacity, W unless lanes are replaced).  Retired lanes give their state at
 * the completion depth (STATIC: at l_max); running lanes give their current state. */
skb_status sinkhorn_batch_potentials(skb_batch *h, float *f, float *g);
skb_status sinkhorn_batch_potentials_f64(skb_batch *h, double *f, double *g);

/* Completion depth l_t (first audited cycle at which the lane passed; Eq. 6) and
 * skb_lane_status per lane, device out [L] (L as above), original lane order; either may be null. */
skb_status sinkhorn_batch_depths(skb_batch *h, int *depth, int *lane_status);

/* Residuals of Eq. 5 measured at the state that was emitted: r_row = |pi 1 - a|_1,
 * r_col = |pi^T 1 - b|_1, device out [L] fp32.  r_col is NaN for a lane that was never
 * sent to the two-sided check (iteration limit without a screen pass). */
skb_status sinkhorn_batch_residuals(skb_batch *h, float *r_row, float *r_col);

/*
 * The coupling applied to caller-supplied values (the plan as an output, Section on endpoints:
 * potentials are the stored result, the plan pi = exp((f + g - C)/eps) of Eq. 3 is implied):
 *     out[t, i, :] = sum_j pi_ij v[t, j, :]
 * for every lane t with the potentials it finished with; v = y gives a_i times the barycentric image
 * of x_i, v = 1 the row marginal.  x, y, eps: the arrays the batch was created from (the batch keeps
 * no lane-ordered copy of them); v [W, m, dv] fp32, out [W, n, dv] fp32, device; 1 <= dv <= 16.
 * Valid once every lane has finished (SKB_ERR_STATE before that, and for batches whose lanes were
 * replaced).  Float64 arithmetic, one pass over all pairs; synchronises to check the state, then
 * enqueues one kernel.
 */
skb_status sinkhorn_batch_apply_plan(skb_batch *h, const void *x, const void *y, const float *eps,
                                     const float *v, int dv, float *out);

/*
 * What the most recent audit measured, per lane still held in a slot (device outs [W], original
 * lane order, any may be null; entries of lanes that have left are not touched): the fused row
 * screen's value r_row, the column residual r_col of screen-positive lanes (NaN otherwise) and
 * whether the lane was screen-positive.  After step(k) these belong to the state after k-1
 * cycles: the screen of a state is a by-product of the NEXT f-leg.  For shadow replays of the
 * audit (Section 5's attribution: does the screen ever hold back a lane the full check would
 * release?).  Kept by the one-launch-per-leg path only: MASKED, STATIC, tensor-core or profiled
 * batches (SKB_ERR_STATE otherwise).  Enqueues one kernel.
 */
skb_status sinkhorn_batch_last_audit(skb_batch *h, float *r_row, float *r_col, int *flagged);

/*
 * Phases of the time model T_active = sum_k c_k(A_k) + H_screen + H_check + H_compact
 * (Section "Hardware realization and break-even", Eq. 11): the update legs are c_k (the row
 * screen rides inside the f-leg, so H_screen has no time of its own), the column check is
 * H_check, planning plus emission/compaction is H_compact.
 */
typedef enum {
    SKB_PHASE_CREATE = 0,       /* set-up kernels of create (always measured)                 */
    SKB_PHASE_F_LEG = 1,        /* f-leg launches, row screen included                        */
    SKB_PHASE_COLUMN_CHECK = 2, /* column half of the two-sided check, flagged lanes only     */
    SKB_PHASE_PLAN = 3,         /* flags -> retire list, hole/filler pairing, counters        */
    SKB_PHASE_EMIT_MOVE = 4,    /* retirees' outputs written, survivors moved into holes       */
    SKB_PHASE_G_LEG = 5,        /* g-leg launches                                             */
    SKB_N_PHASES = 6
} skb_phase;

/*
 * Phase timing on or off (off at creation), only before the first step/drain.  When on, every
 * kernel of every cycle is bracketed by CUDA events on the batch's stream; the kernels of a
 * cycle then run strictly one after the other (normally the next kernel's launch overlaps the
 * current one), so a profiled solve is slower than a plain one and its phases add up to ITS
 * duration.  Events are collected every 16 cycles with a stream synchronisation.
 */
skb_status sinkhorn_batch_set_profiling(skb_batch *h, int on);

/*
 * Work accounting (Eq. 6-8) and the cost record of Eq. 11, host outs, any may be null.
 * Synchronises.
 *   slots      lane-cycles physically executed: sum_k A_k in ACTIVE mode, W*l_max otherwise
 *   cycles     complete cycles executed (l_max)
 *   widths     widths[k-1] = physical width of cycle k, for k = 1..min(cycles, widths_cap)
 *   pair_terms exp-terms evaluated by the update kernel, all passes (legs, look-ahead
 *              screen, column check)
 *   phase_ms   [SKB_N_PHASES] milliseconds per skb_phase summed over the solve so far;
 *              entries other than SKB_PHASE_CREATE are zero unless phase timing is on
 */
skb_status sinkhorn_batch_stats(skb_batch *h, long long *slots, int *cycles, int *widths,
                                int widths_cap, long long *pair_terms, float *phase_ms);

/* Per-cycle update cost c_k of Eq. 11 from a profiled solve: update_ms[k-1] = f-leg + g-leg
 * milliseconds of cycle k (host out, up to cap entries); *count = cycles recorded.  Together
 * with widths[] of sinkhorn_batch_stats this is c_k as a function of the width A_k.
 * Synchronises. */
skb_status sinkhorn_batch_cycle_trace(skb_batch *h, float *update_ms, int cap, int *count);

/* The arithmetic the batch actually runs (skb_compute, never AUTO): what an automatic
 * batch resolved to from its data.  Host out. */
skb_status sinkhorn_batch_arithmetic(skb_batch *h, int *compute);

/*
 * Integrity check of the caller's workspace (a stand-in for a memory checker: every kernel of
 * the path writes through index arithmetic into arrays carved out of one allocation).  Every
 * such array is followed by a guard strip of 256 bytes holding a known pattern, written by
 * create; this call compares all strips and writes to *first_bad (host) the index, in layout
 * order, of the first strip that no longer holds its pattern, or -1 if all are intact.  A
 * damaged strip means a write past the end of the array before it.  May be called at any time
 * after create; launches one small kernel and synchronises the batch's stream.
 * Returns SKB_OK whether or not a strip is damaged; SKB_ERR_NULL / SKB_ERR_CUDA otherwise.
 */
skb_status sinkhorn_batch_check_guards(skb_batch *h, int *first_bad);

/*
 * Self-test of the kernels' failure detection.  The tensor-core kernel synchronises its
 * warps through mbarriers; every such wait has a clock budget, after which the kernel
 * records an error instead of hanging (the host then reports SKB_ERR_CUDA).  This call runs
 * one such wait on a barrier that nothing completes, with the given budget in milliseconds
 * (at ~2 GHz), and writes three ints to out3 (device): 1 if the wait gave up, the abort flag
 * it raised, and the kilo-clocks it spent.  Enqueues only.
 */
skb_status sinkhorn_batch_selftest_bounded_wait(int *out3, float budget_ms, void *stream);

/*
 * Self-test: measured issue rates of the units that bound the update kernels, for quoting a
 * roofline fraction against delivered rather than nominal rates.  Runs four short register-only
 * loops (fp32 FMA, packed fp32x2 FMA, float64 FMA, fp32 ex2) and writes the operations per
 * second of each to ops_per_second[0..3] (host out; an fp32x2 instruction counts as two FMAs).
 * sink: any device float the caller owns (the loops need an address they might write to; they
 * never do).  Synchronises the stream.
 */
skb_status sinkhorn_batch_selftest_unit_rates(double *ops_per_second, float *sink, void *stream);

/* Number of kernels this handle has launched so far (host out). */
skb_status sinkhorn_batch_launch_count(skb_batch *h, long long *launches);

/*
 * Measurement aid: launches the update kernel for one leg (0 = f-leg, 1 = g-leg) `reps`
 * times at the batch's current width, bracketed by CUDA events on the batch's stream, and
 * returns the mean duration per launch in milliseconds (host out).  Call it between cycles
 * (after step, before drain).  The launches are dry runs: all pair work and the row epilogue,
 * but no potential is stored and no residual term added, so a solve continued afterwards
 * gives the same bits as one that was never profiled.  Returns SKB_ERR_STATE when no lane is
 * running any more (the launch would return at once).  Synchronises.
 */
skb_status sinkhorn_batch_profile_update(skb_batch *h, int leg, int reps, float *ms_per_launch);

/*
 * Whole solve from HOST buffers in one call: copies x, y, a, b, eps to the device,
 * creates the batch, drains it, and copies the results back.  Every data pointer here is
 * HOST memory (pinned memory makes the copies asynchronous); outputs may be null.
 * cfg->workspace is still device memory and must hold
 * sinkhorn_batch_host_workspace_bytes(cfg) bytes: the batch's own workspace followed by
 * staging for the inputs and outputs.  Returns after the stream has been synchronised.
 */
size_t sinkhorn_batch_host_workspace_bytes(const skb_config *cfg);
skb_status sinkhorn_batch_solve_host(const void *x, const void *y, const float *a, const float *b,
                                     const float *eps, float tol, const skb_config *cfg,
                                     float *f, float *g, int *depth, int *lane_status,
                                     float *r_row, float *r_col, long long *slots, int *cycles);

void sinkhorn_batch_destroy(skb_batch *h);

/*
 * Row residual of given potentials without any workspace or allocation.  (The paper has no
 * counterpart: this is a library convenience for callers that may not allocate device
 * memory - a host that fixes every component's memory budget at start-up, or a loop that
 * cannot take the device-wide synchronisation of cudaMalloc.)
 *
 * For each lane, r_row = sum_i | sum_j exp((f_i + g_j - |x_i - y_j|^2)/eps) - a_i |, the row
 * half of Eq. 5, in float64 arithmetic.
 *   x [W,n,d], y [W,m,d], a [W,n], eps [W]  fp32, device, row-major
 *   f [W,n], g [W,m]                       float64, device
 *   r_row [W]                              fp32, device out
 *   stream                                 cudaStream_t; the call enqueues and returns
 * The scratch of the reduction is a fixed SKB_STATIC_SCRATCH_BYTES array inside the library
 * image (held by every GPU that loads the library until exit), so W <= SKB_STATIC_MAX_LANES
 * and n <= SKB_STATIC_MAX_ROWS; larger shapes return SKB_ERR_SHAPE.  The call performs no
 * cudaMalloc, cudaFree or other allocating call.  The first call on each device looks the
 * array's device address up (with that device current) and, where the CUDA runtime loads
 * kernels lazily, is also the moment the runtime loads this library's device code onto that
 * device (which reserves device memory for the code and may synchronise): make that first
 * call during warm-up, before any stream capture begins and before memory is frozen.  All
 * calls share the one array: calls whose kernels could overlap on the GPU (different
 * streams, different threads) race and must be ordered by the caller.
 * sinkhorn_row_residual_static_last_error() gives the text of the calling thread's last
 * failed call (empty after a successful one).
 */
#define SKB_STATIC_MAX_LANES 256
#define SKB_STATIC_MAX_ROWS 8192
#define SKB_STATIC_SCRATCH_BYTES (SKB_STATIC_MAX_LANES * (SKB_STATIC_MAX_ROWS / 128) * 8 + SKB_STATIC_MAX_LANES * 4)
skb_status sinkhorn_row_residual_static(const float *x, const float *y, const float *a,
                                        const double *f, const double *g, const float *eps,
                                        int W, int n, int m, int d, float *r_row, void *stream);
const char *sinkhorn_row_residual_static_last_error(void);

/* Host string describing the last error on this handle (or, when h is null, of the calling
 * thread's last failed create or host-buffer solve).  Valid until the next call on the same
 * handle (h null: the next failing create of the same thread). */
const char *sinkhorn_batch_last_error(const skb_batch *h);

#ifdef __cplusplus
}
#endif
#endif /* SINKHORN_BATCH_H */
