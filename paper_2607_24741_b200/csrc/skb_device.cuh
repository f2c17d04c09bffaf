// Device-side state of a Sinkhorn batch and small numeric helpers shared by the kernels.
//
// Internal representation (all lane-indexed arrays are indexed by PHYSICAL SLOT; the
// slot -> original lane map is lane_id[]):
//   s        = log2(e)/eps                      per-lane scale, log2 domain
//   phi, gam = s*f, s*g                          potentials, float64
//   xs, ys   = sqrt(2s)*x, sqrt(2s)*y            coordinates, dimension-major [DP][npad]
//   sqx, sqy = |xs_i|^2/2, |ys_j|^2/2            float64
//   ft, gt   = phi - sqx, gam - sqy              per-point terms streamed by the opposite leg
// so that log2 pi_ij = ft_i + gt_j + xs_i.ys_j  (plan of Eq. 3 with f = eps log u).
// That is the expanded ("dot") form of the cost.  Lanes whose scaled squared radius is so
// large that the expanded form would cancel catastrophically in fp32 use the difference
// form instead: coordinates scaled by sqrt(s), ft/gt hold the high and fl/gl the low part
// of the potentials, and log2 pi_ij = (phi_i + gam_j) - |xs_i - ys_j|^2.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace skb {

enum Leg : int { LEG_F = 0, LEG_G = 1, LEG_V = 2 };
enum Mode : int { MODE_ACTIVE = 0, MODE_MASKED = 1, MODE_STATIC = 2 };
enum LaneStatus : int { LANE_RUNNING = 0, LANE_DONE = 1, LANE_ITER_LIMIT = 2, LANE_NONFINITE = 3 };
enum ErrBits : int { ERR_VALUE = 1, ERR_WAIT = 2 };
enum Form : int { FORM_DOT = 0, FORM_DIFF = 1 };

constexpr float NEG_BIG = -1.0e30f;   // "minus infinity" for padded columns (finite: no NaNs)
constexpr int UPD_THREADS = 128;
constexpr int TC_MAX_SPLIT = 8;      // a row block's columns go to at most this many clusters
constexpr int MAX_CLUSTER_RANKS = 8;  // blocks per cluster (portable limit): row blocks of a lane in the multi-cycle kernels
constexpr double RSUM_SCALE = 17592186044416.0;     // 2^44: unit of the fixed-point residual sums
constexpr double RSUM_ROW_MAX = 4.0;                 // one row's term is clamped here (a whole L1 residual never exceeds 2 near
                                                     // convergence), so fewer than 2^18 rows cannot overflow 64 bits

// Device-resident control block.  Written by the plan kernel (one CTA), read by all.
struct Ctl {
    int n_phys;        // physical width of the next update launch (ACTIVE: survivors; else W)
    int n_running;     // lanes not yet retired
    int cycle;         // completed cycles; the state being audited is the one after `cycle` cycles
    int parity;        // phi[parity] / ft[parity] hold the current row potentials
    int n_retire;      // entries of the retire list written by the last plan
    int emit_parity;   // buffer the retirees' f is emitted from
    int done;          // nothing left to do
    int static_final;  // STATIC: every lane has passed, next audit emits all lanes
    int error;         // sticky ErrBits
    int n_passed;      // STATIC: lanes that have recorded a depth
    int pad0, pad1;
    unsigned long long max_radius_bits;   // largest scaled squared radius over lanes (double bits)
    long long slots;       // lane-cycles physically executed
    long long pair_terms;  // exp terms evaluated by update launches
};

struct Dev {
    int W, n, m, d, np, mp, DP;   // W: slots (lanes held at a time)
    int L;                    // lanes the result buffers hold (> W when finished lanes are replaced by new problems)
    int widths_cap;           // entries of widths[]
    int mode, max_iter, audit_every, xy_bf16, compute_f64, cost_form, tensor;
    int early_exit;           // MASKED only: CTAs of a frozen lane return at once (an extra arm, not the paper's mask control)
    int dry_run;              // measurement launches: a leg computes everything but stores no potential and adds no residual term
    int audit_initial;        // warm proposals: the state before the first cycle is audited too (a lane may retire at depth 0)
    double form_threshold;    // scaled squared radius above which a lane uses the difference form
    double tol_screen, tol_stop;
    // slabs by slot
    void *xs, *ys;            // [W][DP][np|mp]   T   (SIMT kernels)
    void *xb, *yb;            // bf16 copies tiled [W][128-point tile][64-dim chunk][128][64] (tensor-core kernel)
    void *ft[2];              // [W][np]          T
    void *gt;                 // [W][mp]          T
    void *fl[2], *gl;         // low parts of the potentials (difference form only)
    double *center;           // [W][DP] joint centroid of the lane's two clouds
    double *sqx, *sqy;        // [W][np], [W][mp]
    double *la2, *lb2;        // log2 a, log2 b
    double *wa, *wb;          // a, b
    double *phi[2];           // [W][np]
    double *gam;              // [W][mp]
    // per-slot scalars
    double *scale;            // s
    int *lane_id;
    int *start;               // cycle count of the batch when the lane in the slot came in (0 for the first W lanes)
    int *form;                // Form per slot
    int *state;               // MASKED: frozen; STATIC: passed
    int *flag;                // screen-positive at this audit
    int *verdict;             // two-sided check passed
    int *nonfinite;
    // multi-cycle launches: cycle count + 1 at which the lane in the slot left inside the launch
    // (0 = still running), and the column checks it ran
    int *ret_at, *n_checks;
    // guard band (float64 escalation of a near-threshold screen): raw copies of the inputs by slot,
    // the relative half-width of the band (0 = off), the escalated row residual as a fixed-point
    // sum and whether it was taken at this audit
    void *xraw, *yraw;        // [W][n][d], [W][m][d] in the inputs' own type, each slot padded to a multiple of 16 bytes
    size_t xraw_stride, yraw_stride;   // bytes per slot
    double guard;
    unsigned long long *rsum_row64;
    int *esc;
    double *rrow, *rcol;      // residuals of the audited state
    // marginal residuals of the audited state as fixed-point sums (units of 2^-44): every row block
    // adds its part with one integer atomic, so the total is exact and independent of the order
    // of arrival; the plan kernel turns them into rrow / rcol / flag / verdict and clears them
    unsigned long long *rsum_row, *rsum_col;
    // tensor path for d > 256: arrival word of a row block whose column tiles were shared out among
    // clusters, and every unit's row results [W][row block][TC_MAX_SPLIT][column half][128]
    unsigned *tc_cnt;
    float *tc_pm;
    double *tc_ps;
    // retire / move lists (plan -> emit_move)
    int *ret_slot, *ret_lane, *ret_src;
    double *ret_scale;
    int *hole_list, *fill_list;
    // results by original lane
    double *f_out, *g_out;    // [W][n], [W][m]  potentials in the caller's units
    int *depth, *status, *emitted;
    double *res_row, *res_col;
    int *widths;              // [max_iter + 2]
    int *guard_bad;           // result word of the guard-strip check
    Ctl *ctl;
};

// Guard strips of the workspace: 256 bytes of a known pattern after every array the library carves
// out of the caller's workspace, so that a write past the end of an array is found, on request,
// instead of silently landing in its neighbour.  Offsets in units of 256 bytes from the workspace.
constexpr int GUARD_STRIP_BYTES = 256;
constexpr int MAX_GUARD_STRIPS = 96;
struct GuardList {
    int count;
    unsigned off256[MAX_GUARD_STRIPS];
};

// Raw coordinate of the inputs' own storage type (fp32, or bf16 widened exactly).
__device__ __forceinline__ float load_raw(const Dev &P, const void *base, size_t idx)
{
    if (P.xy_bf16) return __uint_as_float(((unsigned)reinterpret_cast<const unsigned short *>(base)[idx]) << 16);
    return reinterpret_cast<const float *>(base)[idx];
}

// Guard band around the thresholds (the paper's stress test of near-threshold accept decisions,
// Section 5: an outward guard with float64 escalation).  A screen value this close to a threshold
// is within the evaluation error of the fp32 exponentials, so the decision is taken from a float64
// re-evaluation instead.
// The band is relative to the threshold with an absolute floor: the fused screen's error is a few 1e-8
// absolute whatever the tolerance (measured), i.e. 3e-5 of a tolerance of 1e-3 but 3e-4 of 1e-4.
constexpr double GUARD_ABS_FLOOR = 1.0e-7;
__device__ __forceinline__ bool in_guard_band(const Dev &P, const double rr)
{
    return P.guard > 0.0 && (fabs(rr - P.tol_screen) <= fmax(P.guard * P.tol_screen, GUARD_ABS_FLOOR) ||
                             fabs(rr - P.tol_stop) <= fmax(P.guard * P.tol_stop, GUARD_ABS_FLOOR));
}

// One row's term |sum_j pi_ij - a_i| of the row residual (Eq. 5), from the raw inputs and the
// float64 potentials, float64 throughout (difference-form cost, software exp2): the plain
// definition, independent of the update kernels' layouts and arithmetic.  One WARP per row: lane l
// takes the columns l, l + 32, ... with its own running maximum and sum, and the 32 pairs are merged
// by xor-shuffles (every lane returns the term).  phi: the row's potential (log2 units); the column
// potentials are read from global memory past L1, because inside a multi-cycle launch other blocks of
// the cluster have written them.
template <bool VEC = false>
__device__ __forceinline__ double direct_row_term_warp(const Dev &P, const int slot, const int i, const double phi)
{
    const int lane = threadIdx.x & 31;
    const double s = P.scale[slot];
    const double *gam = P.gam + (size_t)slot * P.mp;
    const void *xl = (const char *)P.xraw + (size_t)slot * P.xraw_stride;
    const void *yl = (const char *)P.yraw + (size_t)slot * P.yraw_stride;
    const size_t xb = (size_t)i * P.d;
    double mx = -1.0e300, sum = 0.0;
    // four columns per lane and step: their cost chains and exponentials are independent, which is
    // what keeps the float64 pipe busy at the few warps an escalation runs on
    constexpr int U = 4;
    for (int j0 = lane; j0 < P.m; j0 += 32 * U) {
        size_t yb[U];
        double c[U], gj[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int j = j0 + 32 * u;
            const int jc = j < P.m ? j : P.m - 1;          // clamped: loads stay inside the lane, the term is dropped below
            yb[u] = (size_t)jc * P.d;
            gj[u] = __ldcg(gam + jc);
            c[u] = 0.0;
        }
        if (VEC && P.xy_bf16 && (P.d & 7) == 0) {       // VEC: only the stand-alone pool kernel carries this path
            // deep bf16 lanes: eight dimensions per 16-byte load (same operations in the same order)
            const unsigned short *x16 = reinterpret_cast<const unsigned short *>(xl);
            const unsigned short *y16 = reinterpret_cast<const unsigned short *>(yl);
            for (int k = 0; k < P.d; k += 8) {
                const uint4 xv = *reinterpret_cast<const uint4 *>(x16 + xb + k);
                const unsigned xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint4 yv = *reinterpret_cast<const uint4 *>(y16 + yb[u] + k);
                    const unsigned yw[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const double t0 = (double)__uint_as_float(xw[e] << 16) - (double)__uint_as_float(yw[e] << 16);
                        c[u] = fma(t0, t0, c[u]);
                        const double t1 = (double)__uint_as_float(xw[e] & 0xffff0000u) - (double)__uint_as_float(yw[e] & 0xffff0000u);
                        c[u] = fma(t1, t1, c[u]);
                    }
                }
            }
        } else {
            for (int k = 0; k < P.d; ++k) {
                const double xk = (double)load_raw(P, xl, xb + k);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const double t = xk - (double)load_raw(P, yl, yb[u] + k);
                    c[u] = fma(t, t, c[u]);
                }
            }
        }
        double v[U], mn = mx;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            v[u] = (j0 + 32 * u < P.m) ? phi + gj[u] - s * c[u] : -1.0e300;
            mn = fmax(mn, v[u]);
        }
        double add = 0.0;
#pragma unroll
        for (int u = 0; u < U; ++u) add += (j0 + 32 * u < P.m) ? exp2(v[u] - mn) : 0.0;
        sum = sum * exp2(mx - mn) + add;
        mx = mn;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const double mo = __shfl_xor_sync(0xffffffffu, mx, off);
        const double so = __shfl_xor_sync(0xffffffffu, sum, off);
        const double mn = fmax(mx, mo);
        sum = sum * exp2(mx - mn) + so * exp2(mo - mn);      // a lane without columns carries (-1e300, 0): its factor underflows to 0
        mx = mn;
    }
    return fabs(exp2(mx) * sum - P.wa[(size_t)slot * P.np + i]);
}

// Rows of a lane for one block of NW warps, one warp per row: warp w takes the rows row_first + w,
// row_first + w + stride, ... below row_end.  Returns this block's exact fixed-point part of the
// float64 row residual (valid in thread 0) and whether a term was not finite.  pot[i - pot_first] is
// row i's potential.
template <int NW, bool VEC = false>
__device__ __forceinline__ unsigned long long direct_rows_block(const Dev &P, const int slot, const int row_first,
                                                                const int stride, const int row_end, const double *pot,
                                                                const int pot_first, unsigned long long *red, int *nf)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned long long part = 0ull;
    int bad = 0;
    for (int i = row_first + warp; i < row_end; i += stride) {
        const double term = direct_row_term_warp<VEC>(P, slot, i, pot[i - pot_first]);
        if (!isfinite(term)) bad = 1;
        else if (lane == 0) part += __double2ull_rn(fmin(term, RSUM_ROW_MAX) * RSUM_SCALE);
    }
    bad = __syncthreads_or(bad);
    if (lane == 0) red[warp] = part;
    __syncthreads();
    unsigned long long sum = 0ull;
    if (threadIdx.x == 0) for (int w = 0; w < NW; ++w) sum += red[w];
    __syncthreads();
    *nf = bad;
    return sum;
}

// Is the state of a lane that came in at batch cycle `start` audited when the batch has completed
// `cycle` cycles?  Audits sit on the BATCH's grid (every audit_every-th cycle) and need at least one
// cycle of the lane's own; a warm proposal may be audited before its first cycle.
__device__ __forceinline__ bool lane_audited(const Dev &P, const int cycle, const int start)
{
    return (cycle - start >= 1 && (cycle % P.audit_every) == 0) || (cycle == 0 && P.audit_initial);
}

// The row residual a lane's decisions are taken from: the escalated value if one was taken.
__device__ __forceinline__ double lane_row_residual(const Dev &P, const int slot)
{
    return (double)(P.esc[slot] ? P.rsum_row64[slot] : P.rsum_row[slot]) * (1.0 / RSUM_SCALE);
}

// Screen verdict of a lane from its accumulated row residual: the same predicate for the column
// check (which lanes to visit) and for the planner (which lanes may retire).
__device__ __forceinline__ bool lane_flag(const Dev &P, const Ctl &c, const int slot)
{
    const bool passed = P.state[slot] != 0;                  // MASKED: frozen; STATIC: already passed
    const bool audited = lane_audited(P, c.cycle, P.start[slot]);
    const bool live = !(passed && (P.mode == MODE_MASKED || P.mode == MODE_STATIC));
    return audited && live && !P.nonfinite[slot] && lane_row_residual(P, slot) <= P.tol_screen;
}

// Which lanes the column check visits: the screen-positive ones and, with a guard band, every lane
// whose screen value lies inside the band - its decision comes from the float64 re-evaluation that
// other blocks of the same launch are computing, so the column residual is measured in case it passes.
__device__ __forceinline__ bool lane_needs_column_check(const Dev &P, const Ctl &c, const int slot)
{
    if (lane_flag(P, c, slot)) return true;
    if (!(P.guard > 0.0)) return false;
    const bool passed = P.state[slot] != 0;
    const bool audited = lane_audited(P, c.cycle, P.start[slot]);
    const bool live = !(passed && (P.mode == MODE_MASKED || P.mode == MODE_STATIC));
    return audited && live && !P.nonfinite[slot] && in_guard_band(P, (double)P.rsum_row[slot] * (1.0 / RSUM_SCALE));
}

__device__ __forceinline__ float ex2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float ex2_t(float x) { return ex2_fast(x); }
__device__ __forceinline__ double ex2_t(double x) { return exp2(x); }

// Programmatic dependent launch: wait until the kernels this launch depends on have completed
// and their writes are visible, then let the NEXT kernel in the stream start launching (it
// blocks at its own wait), so launch latency overlaps execution.  A no-op for plain launches.
__device__ __forceinline__ void pdl_enter()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

}  // namespace skb
