// Matrix-free Sinkhorn half-step (Eq. 3 in log form) as one streaming kernel.
//
// One launch serves every active lane (grid.y = physical width, grid.x = row blocks):
// the candidate axis of Eq. 2 is a grid axis and nothing is reduced across lanes.
//
// For a row point i of lane t the kernel evaluates, over all column points j,
//     L_i = log2 sum_j 2^(arg_ij)
// as an online max / sum-of-exp2 reduction: the n x m matrix is never stored.  Column
// tiles are staged in shared memory by 16-byte cp.async copies from a dimension-major
// layout; a thread keeps R rows in registers and walks 4 adjacent columns per step; with
// CS > 1 the columns of a tile are split over CS neighbouring lanes of the warp and the
// (max, sum) pairs are merged by xor-shuffles at the end.
//
// Two forms of arg_ij, chosen per lane when the batch is created:
//   dot   arg_ij = ct_j + r_i . c_j            (d FMA per pair; ct = potential - |c_j|^2/2)
//   diff  arg_ij = (ph_i + ch_j) + cl_j - |r_i - c_j|^2   (2d + 2 per pair; ph, ch are the
//         fp32 high parts of the row and column potentials, cl the column's low part, and
//         the row's own rounding error is removed in float64 afterwards).  It is used when
//         the expanded form would cancel catastrophically in fp32.
//
// Leg-specific epilogues (float64, one per row):
//   LEG_F  phi_new from L;  also the row marginal of the state BEFORE this leg,
//          sum_j pi_ij = a_i 2^(phi_old - phi_new), which is the one-sided row screen of
//          Section "Screen, verify, and compact" obtained for free.
//   LEG_G  gam_new from L  (after it the column marginal equals b, Eq. 4).
//   LEG_V  column marginal of the audited state for screen-positive lanes only,
//          the second half of the two-sided check (Eq. 5).
// The per-CTA L1 partial sums go to scratch; the last CTA of a lane adds them in a fixed
// order and writes the lane's residual and its one flag (screen-positive / verdict).
#pragma once
#include "skb_device.cuh"

namespace skb {

template <typename T, int XF> struct SumType { using type = T; };
template <> struct SumType<double, 1> { using type = float; };

template <int CS> struct TileCols { static constexpr int value = (CS <= 4) ? 128 : (CS == 8 ? 256 : 512); };

__device__ __forceinline__ void lds4(const float *p, float (&v)[4])
{
    float4 t = *reinterpret_cast<const float4 *>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void lds4(const double *p, double (&v)[4])
{
    double2 t0 = *reinterpret_cast<const double2 *>(p);
    double2 t1 = *reinterpret_cast<const double2 *>(p + 2);
    v[0] = t0.x; v[1] = t0.y; v[2] = t1.x; v[3] = t1.y;
}

// Streams every column tile of one lane past the CTA's rows and leaves, per row of this
// thread, the running maximum md[r] and the sum sd[r] of 2^(arg - md[r]) over the columns
// this thread visited.
template <typename T, int DP, int R, int CS, int FORM, int XF>
__device__ __forceinline__ void stream_columns(T *sm, const T *colc, const T *colt, const T *coll,
                                               const int cp, const int ncols, const T (&xr)[R][DP],
                                               const T (&ph)[R], const int tid, const int cs,
                                               double (&md)[R], double (&sd)[R])
{
    constexpr int TJ = TileCols<CS>::value;
    constexpr int STEPS = TJ / (4 * CS);
    constexpr int EPC = 16 / (int)sizeof(T);
    constexpr int NR = DP + 1 + (FORM == FORM_DIFF ? 1 : 0);   // rows of a stage
    constexpr int STAGE = (DP + 2) * TJ;
    constexpr int CPR = TJ / EPC;

    // XF = 1: the exponentials run on the fp32 special-function unit even when the
    // arguments are float64 ("mixed" arithmetic); the tile sum is then fp32 as well
    using TS = typename SumType<T, XF>::type;
    T mx[R];
    TS ts[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { mx[r] = T(NEG_BIG); ts[r] = TS(0); sd[r] = 0.0; }

    const int ntiles = (ncols + TJ - 1) / TJ;
    auto load_tile = [&](int t, int stage) {
        T *dst = sm + stage * STAGE;
        const int j0 = t * TJ;
        for (int ch = tid; ch < NR * CPR; ch += UPD_THREADS) {
            const int k = ch / CPR, j = j0 + (ch % CPR) * EPC;
            T *d = dst + k * TJ + (ch % CPR) * EPC;
            if (j < cp) {
                const T *src = (k < DP) ? colc + (size_t)k * cp + j : (k == DP ? colt + j : coll + j);
                cp_async16(d, src);
            } else {
                // columns past the padded end: zero coordinates, "minus infinity" term
                const T fill = (k == DP) ? T(NEG_BIG) : T(0);
#pragma unroll
                for (int e = 0; e < EPC; ++e) d[e] = fill;
            }
        }
    };

    load_tile(0, 0);
    cp_async_commit();
    for (int t = 0; t < ntiles; ++t) {
        if (t + 1 < ntiles) {
            load_tile(t + 1, (t + 1) & 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const T *st = sm + (t & 1) * STAGE;
#pragma unroll 2
        for (int q = 0; q < STEPS; ++q) {
            const int jj = (q * CS + cs) * 4;
            T acc[R][4];
            T ct[4];
            lds4(st + DP * TJ + jj, ct);
            if (FORM == FORM_DOT) {
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[r][e] = ct[e];
#pragma unroll
                for (int k = 0; k < DP; ++k) {
                    T yv[4];
                    lds4(st + k * TJ + jj, yv);
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[r][e] = fma(xr[r][k], yv[e], acc[r][e]);
                }
            } else {
                T cl[4];
                lds4(st + (DP + 1) * TJ + jj, cl);
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[r][e] = cl[e];
#pragma unroll
                for (int k = 0; k < DP; ++k) {
                    T yv[4];
                    lds4(st + k * TJ + jj, yv);
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const T dk = xr[r][k] - yv[e];
                            acc[r][e] = fma(-dk, dk, acc[r][e]);
                        }
                }
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[r][e] += (ph[r] + ct[e]);
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const T mt = fmax(fmax(acc[r][0], acc[r][1]), fmax(acc[r][2], acc[r][3]));
                if (mt > mx[r] + T(8)) {           // lazy rescale: terms stay below 2^8
                    const TS fac = ex2_t((TS)(mx[r] - mt));
                    ts[r] *= fac;
                    sd[r] *= (double)fac;
                    mx[r] = mt;
                }
                ts[r] += (ex2_t((TS)(acc[r][0] - mx[r])) + ex2_t((TS)(acc[r][1] - mx[r]))) +
                         (ex2_t((TS)(acc[r][2] - mx[r])) + ex2_t((TS)(acc[r][3] - mx[r])));
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) { sd[r] += (double)ts[r]; ts[r] = TS(0); }
        __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < R; ++r) md[r] = (double)mx[r];
}

template <typename T, int DP, int R, int CS, int XF>
__global__ void __launch_bounds__(UPD_THREADS) update_kernel(const Dev P, const int leg)
{
    constexpr int RG = 32 / CS;                  // row groups per warp
    constexpr int RW = R * RG;                   // rows per warp
    constexpr int RB = (UPD_THREADS / 32) * RW;  // rows per CTA

    extern __shared__ __align__(16) unsigned char smem_raw[];
    T *sm = reinterpret_cast<T *>(smem_raw);
    __shared__ double red[UPD_THREADS / 32];
    __shared__ int is_last;

    const Ctl c = *P.ctl;
    if (c.done) return;
    const int slot = blockIdx.y;
    if (slot >= c.n_phys) return;
    if (leg != LEG_V && c.static_final) return;
    if (leg == LEG_V && !(c.static_final || P.flag[slot])) return;

    // roles: rows are x-points for the f-leg, y-points otherwise
    const bool rows_x = (leg == LEG_F);
    const int nrows = rows_x ? P.n : P.m, rp = rows_x ? P.np : P.mp;
    const int ncols = rows_x ? P.m : P.n, cp = rows_x ? P.mp : P.np;
    if ((int)blockIdx.x * RB >= nrows) return;
    const int form = (sizeof(T) == 8) ? (int)FORM_DOT : P.form[slot];   // float64 arguments never need the difference form
    const T *rowc = reinterpret_cast<const T *>(rows_x ? P.xs : P.ys) + (size_t)slot * DP * rp;
    const T *colc = reinterpret_cast<const T *>(rows_x ? P.ys : P.xs) + (size_t)slot * DP * cp;
    const T *colt = rows_x ? reinterpret_cast<const T *>(P.gt) + (size_t)slot * cp
                           : reinterpret_cast<const T *>(P.ft[c.parity]) + (size_t)slot * cp;
    const T *coll = rows_x ? reinterpret_cast<const T *>(P.gl) + (size_t)slot * cp
                           : reinterpret_cast<const T *>(P.fl[c.parity]) + (size_t)slot * cp;
    // potential the rows carry into this leg (shift of the difference form, screen reference)
    const double *prow = (rows_x ? P.phi[c.parity] : P.gam) + (size_t)slot * rp;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cs = lane % CS, rg = lane / CS;
    const int row0 = blockIdx.x * RB + warp * RW + rg;   // row r of this thread: row0 + r*RG

    T xr[R][DP], ph[R];
    double pold[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int i = row0 + r * RG;
#pragma unroll
        for (int k = 0; k < DP; ++k) xr[r][k] = (i < nrows) ? rowc[(size_t)k * rp + i] : T(0);
        pold[r] = (i < nrows) ? prow[i] : 0.0;
        ph[r] = (T)pold[r];
    }

    double md[R], sd[R];
    if (form == FORM_DOT)
        stream_columns<T, DP, R, CS, FORM_DOT, XF>(sm, colc, colt, coll, cp, ncols, xr, ph, tid, cs, md, sd);
    else
        stream_columns<T, DP, R, CS, FORM_DIFF, XF>(sm, colc, colt, coll, cp, ncols, xr, ph, tid, cs, md, sd);

    // merge the CS column splits of each row (xor-shuffle online logsumexp)
#pragma unroll
    for (int off = 1; off < CS; off <<= 1) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const double mo = __shfl_xor_sync(0xffffffffu, md[r], off);
            const double so = __shfl_xor_sync(0xffffffffu, sd[r], off);
            const double mn = fmax(md[r], mo);
            sd[r] = sd[r] * exp2(md[r] - mn) + so * exp2(mo - mn);
            md[r] = mn;
        }
    }

    // epilogue (float64 per row)
    const bool frozen = (P.mode == MODE_MASKED) && P.state[slot] != 0;
    const bool writes = !frozen && leg != LEG_V;
    double term_sum = 0.0;
    if (cs == 0) {
        const size_t rbase = (size_t)slot * rp;
        const double *sq = (rows_x ? P.sqx : P.sqy) + rbase;
        const double *lw = (rows_x ? P.la2 : P.lb2) + rbase;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int i = row0 + r * RG;
            if (i >= nrows) continue;
            const double L = md[r] + log2(sd[r]);
            // log2 of this row's marginal under the potentials the leg started from, and the
            // updated potential that makes the marginal equal to the weight (Eq. 3)
            double lmarg, pnew;
            if (form == FORM_DOT) {
                pnew = lw[i] + sq[i] - L;
                lmarg = lw[i] + pold[r] - pnew;
            } else {
                lmarg = L - ((double)ph[r] - pold[r]);
                pnew = pold[r] + (lw[i] - lmarg);
            }
            if (leg != LEG_G) term_sum += exp2(lw[i]) * fabs(expm1((lmarg - lw[i]) * 0.6931471805599453));
            if (writes) {
                T hi, lo;
                if (form == FORM_DOT) { hi = (T)(pnew - sq[i]); lo = T(0); }
                else { hi = (T)pnew; lo = (T)(pnew - (double)hi); }
                if (leg == LEG_F) {
                    P.phi[c.parity ^ 1][rbase + i] = pnew;
                    reinterpret_cast<T *>(P.ft[c.parity ^ 1])[rbase + i] = hi;
                    reinterpret_cast<T *>(P.fl[c.parity ^ 1])[rbase + i] = lo;
                } else {
                    P.gam[rbase + i] = pnew;
                    reinterpret_cast<T *>(P.gt)[rbase + i] = hi;
                    reinterpret_cast<T *>(P.gl)[rbase + i] = lo;
                }
            }
        }
    }
    if (leg == LEG_G) return;

    // fused marginal-residual reduction -> one flag per lane (fixed summation order)
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) term_sum += __shfl_down_sync(0xffffffffu, term_sum, off);
    if (lane == 0) red[warp] = term_sum;
    __syncthreads();
    double *parts = (leg == LEG_F ? P.part_row : P.part_col) + (size_t)slot * MAX_PARTS;
    unsigned *cnt = (leg == LEG_F ? P.cnt_row : P.cnt_col) + slot;
    const int nblk = (nrows + RB - 1) / RB;
    if (tid == 0) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < UPD_THREADS / 32; ++w) s += red[w];
        parts[blockIdx.x] = s;
        __threadfence();
        const unsigned ticket = atomicAdd(cnt, 1u);
        is_last = (ticket == (unsigned)(nblk - 1));
    }
    __syncthreads();
    if (!is_last || tid != 0) return;
    __threadfence();
    double tot = 0.0;
    for (int b = 0; b < nblk; ++b) tot += reinterpret_cast<volatile double *>(parts)[b];
    *cnt = 0u;
    const bool finite = isfinite(tot);
    if (leg == LEG_F) {
        P.rrow[slot] = tot;
        const bool audited = c.cycle >= 1 && (c.cycle % P.audit_every) == 0;
        const bool live = !frozen && !(P.mode == MODE_STATIC && P.state[slot] != 0);
        P.flag[slot] = (audited && live && finite && tot <= P.tol_screen) ? 1 : 0;
        if (!finite && !frozen) P.nonfinite[slot] = 1;
    } else {
        P.rcol[slot] = tot;
        const double two = fmax(P.rrow[slot], tot);
        P.verdict[slot] = (finite && two <= P.tol_stop) ? 1 : 0;
        if (!finite) P.nonfinite[slot] = 1;
    }
}

}  // namespace skb
