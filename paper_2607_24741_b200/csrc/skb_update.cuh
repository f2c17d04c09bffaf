// Matrix-free Sinkhorn half-step (Eq. 3 in log form) as one streaming kernel.
//
// One launch serves every active lane (grid.y = physical width, grid.x = row blocks):
// the candidate axis of Eq. 2 is a grid axis and nothing is reduced across lanes.
//
// For a row point i of lane t the kernel evaluates, over all column points j,
//     L_i = log2 sum_j 2^(arg_ij)
// as an online max / sum-of-exp2 reduction: the n x m matrix is never stored.  Column
// tiles are staged in shared memory by 16-byte cp.async copies from a dimension-major
// layout; a thread keeps R rows in registers and walks a group of adjacent columns per
// step; with CS > 1 the column groups of a tile are dealt round-robin to CS neighbouring
// lanes of the warp and the (max, sum) pairs are merged by xor-shuffles at the end.
// The reference point (running maximum) is kept integer-valued, so every rescale is an exact
// power of two; it only moves when a step's sum of exponentials says it must.
//
// Arithmetic of arg_ij:
//   fp32, dot form   arg = ct_j + r_i . c_j, packed two columns at a time (fma.rn.f32x2);
//   fp32, diff form  arg = (ph_i + ch_j) + (cl_j - |r_i - c_j|^2), for lanes whose scaled
//                    radius makes the expanded form cancel catastrophically in fp32
//                    (ph, ch: fp32 high parts of the potentials, cl: the column's low part;
//                    the row's own rounding error is removed in float64 afterwards);
//   float64          arg = ct_j + r_i . c_j on the FP64 pipe, with the exponentials either
//                    on the fp32 special-function unit ("mixed") or in software (validation).
//
// Leg-specific epilogues (float64, one thread per row, rows handed over through shared
// memory so that no lane repeats another's work):
//   LEG_F  phi_new from L;  also the row marginal of the state BEFORE this leg,
//          sum_j pi_ij = a_i 2^(phi_old - phi_new), which is the one-sided row screen of
//          Section "Screen, verify, and compact" obtained for free.
//   LEG_G  gam_new from L  (after it the column marginal equals b, Eq. 4).
//   LEG_V  column marginal of the audited state for screen-positive lanes only,
//          the second half of the two-sided check (Eq. 5).
// The rows' L1 terms are summed in fixed point (exactly, whatever the grouping and order) into one
// total per lane; the plan kernel turns the totals into the lane's residual, its one flag
// (screen-positive) and the verdict, and the column-check leg reads the same flag predicate.
#pragma once
#include "skb_device.cuh"

namespace skb {

typedef unsigned long long u64;

// Register tile of one thread: R rows held for the whole kernel x CW adjacent columns per step.
// More rows per thread means fewer shared-memory bytes per pair; the limit is the register file.
template <typename T, int DP> struct Tune;
#ifndef SKB_F32_R16
#define SKB_F32_R16 4
#endif
#ifndef SKB_F32_CW16
#define SKB_F32_CW16 4
#endif
#ifndef SKB_UNROLL_Q
#define SKB_UNROLL_Q 1
#endif
template <int DP> struct Tune<float, DP> {
    static constexpr int R = DP <= 8 ? 4 : (DP == 16 ? SKB_F32_R16 : 2);
    static constexpr int CW = DP <= 8 ? 8 : (DP == 16 ? SKB_F32_CW16 : 4);
};
#ifndef SKB_F64_R
#define SKB_F64_R 2
#endif
#ifndef SKB_F64_CW
#define SKB_F64_CW 4
#endif
template <int DP> struct Tune<double, DP> {
    static constexpr int R = DP <= 8 ? SKB_F64_R : 2;
    static constexpr int CW = DP <= 8 ? SKB_F64_CW : 4;
};

// Columns per shared-memory tile: at least two steps, and enough of them between the two barriers
// of a tile that the warps of a CTA drift apart (the special-function unit idles when they all do
// FMAs at once); bounded by the shared memory the double-buffered tile may take.
#ifndef SKB_TJ_SMALL
#define SKB_TJ_SMALL 512
#endif
template <typename T, int DP, int CS> struct TileCols {
    static constexpr int wish = sizeof(T) == 8 ? 128 : (DP <= 4 ? SKB_TJ_SMALL : (DP <= 16 ? 256 : 128));
    static constexpr int value = (Tune<T, DP>::CW * CS * 2 > wish) ? Tune<T, DP>::CW * CS * 2 : wish;
};

__device__ __forceinline__ u64 pack2(float lo, float hi)
{
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c)
{
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b)
{
    u64 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ u64 sub2(u64 a, u64 b)
{
    u64 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// 2^k for an integer-valued k <= 0 (exact; flushes to 0 below the normal range)
__device__ __forceinline__ float pow2i(float k)
{
    const int e = (int)fmaxf(k, -127.0f) + 127;
    return __int_as_float(e << 23);
}

// R consecutive values as one (or two) aligned vector loads; zeros when `ok` is false.
template <typename T, int R>
__device__ __forceinline__ void load_rows(const T *p, const bool ok, T (&v)[R])
{
    constexpr int BYTES = R * (int)sizeof(T);
    if (!ok) {
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = T(0);
        return;
    }
    if constexpr (BYTES == 4) {
        v[0] = p[0];
    } else if constexpr (BYTES == 8) {
        const uint2 t = *reinterpret_cast<const uint2 *>(p);
        memcpy(v, &t, 8);
    } else if constexpr (BYTES == 16) {
        const uint4 t = *reinterpret_cast<const uint4 *>(p);
        memcpy(v, &t, 16);
    } else {
        static_assert(BYTES == 32, "unsupported row vector");
        const uint4 t0 = *reinterpret_cast<const uint4 *>(p);
        const uint4 t1 = *reinterpret_cast<const uint4 *>(reinterpret_cast<const char *>(p) + 16);
        memcpy(v, &t0, 16);
        memcpy(reinterpret_cast<char *>(v) + 16, &t1, 16);
    }
}

// Column-tile loader shared by all arithmetic flavours: NR rows of TJ elements per stage.
template <typename T, int DP, int TJ, int NR>
__device__ __forceinline__ void load_tile(T *dst, const T *colc, const T *colt, const T *coll,
                                          const int cp, const int j0, const int tid)
{
    constexpr int EPC = 16 / (int)sizeof(T);
    constexpr int CPR = TJ / EPC;
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
}

// ------------------------------------------------------------------ fp32, packed pairs
// Leaves per row the integer-valued maximum mx[r] and sd[r] = sum 2^(arg - mx[r]) over the
// columns this thread visited.
template <int DP, int CS, int FORM, int R>
__device__ __forceinline__ void stream_f32(float *sm, const float *colc, const float *colt, const float *coll,
                                           const int cp, const int ncols,
                                           const float (&xrow)[R][DP],
                                           const float (&ph)[R], const int tid, const int cs,
                                           float (&mx)[R], double (&sd)[R])
{
    constexpr int CW = Tune<float, DP>::CW;
    constexpr int NP = CW / 2;                       // packed column pairs per step
    constexpr int TJ = TileCols<float, DP, CS>::value;
    constexpr int STEPS = TJ / (CW * CS);
    constexpr int NR = DP + 1 + (FORM == FORM_DIFF ? 1 : 0);
    constexpr int STAGE = (DP + 2) * TJ;

    u64 xd[R][DP];                       // each row coordinate duplicated into both halves
    u64 phd[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int k = 0; k < DP; ++k) xd[r][k] = pack2(xrow[r][k], xrow[r][k]);
        phd[r] = pack2(ph[r], ph[r]);
    }
    u64 ts[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { mx[r] = NEG_BIG; ts[r] = 0ull; sd[r] = 0.0; }

    const int ntiles = (ncols + TJ - 1) / TJ;
    load_tile<float, DP, TJ, NR>(sm, colc, colt, coll, cp, 0, tid);
    cp_async_commit();
    for (int t = 0; t < ntiles; ++t) {
        if (t + 1 < ntiles) {
            load_tile<float, DP, TJ, NR>(sm + ((t + 1) & 1) * STAGE, colc, colt, coll, cp, (t + 1) * TJ, tid);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const float *st = sm + (t & 1) * STAGE;
        constexpr int UQ = SKB_UNROLL_Q;
#pragma unroll UQ
        for (int q = 0; q < STEPS; ++q) {
            const int jj = (q * CS + cs) * CW;
            u64 acc[R][NP];
            u64 ct[NP];
#pragma unroll
            for (int h = 0; h < NP / 2; ++h) {
                const ulonglong2 c = *reinterpret_cast<const ulonglong2 *>(st + DP * TJ + jj + 4 * h);
                ct[2 * h] = c.x; ct[2 * h + 1] = c.y;
            }
            if (FORM == FORM_DOT) {
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int p = 0; p < NP; ++p) acc[r][p] = ct[p];
#pragma unroll
                for (int k = 0; k < DP; ++k) {
                    u64 y[NP];
#pragma unroll
                    for (int h = 0; h < NP / 2; ++h) {
                        const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(st + k * TJ + jj + 4 * h);
                        y[2 * h] = v.x; y[2 * h + 1] = v.y;
                    }
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int p = 0; p < NP; ++p) acc[r][p] = fma2(xd[r][k], y[p], acc[r][p]);
                }
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int p = 0; p < NP; ++p) acc[r][p] = 0ull;          // |r - c|^2 so far
#pragma unroll
                for (int k = 0; k < DP; ++k) {
                    u64 y[NP];
#pragma unroll
                    for (int h = 0; h < NP / 2; ++h) {
                        const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(st + k * TJ + jj + 4 * h);
                        y[2 * h] = v.x; y[2 * h + 1] = v.y;
                    }
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int p = 0; p < NP; ++p) {
                            const u64 dk = sub2(xd[r][k], y[p]);
                            acc[r][p] = fma2(dk, dk, acc[r][p]);
                        }
                }
                u64 cl[NP];
#pragma unroll
                for (int h = 0; h < NP / 2; ++h) {
                    const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(st + (DP + 1) * TJ + jj + 4 * h);
                    cl[2 * h] = v.x; cl[2 * h + 1] = v.y;
                }
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int p = 0; p < NP; ++p) acc[r][p] = add2(add2(phd[r], ct[p]), sub2(cl[p], acc[r][p]));
            }
            // Exponentials against the reference as it stands; only their sum is tested.  A sum
            // above 2^10 (an argument more than ~8 above the reference, which would cost exponent
            // accuracy; a reference of minus infinity gives an infinite sum) sends the step
            // through the exact path: maxima, integer-valued new references, exact rescale.
            u64 es[R];
            bool grow = false;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const u64 mm = pack2(mx[r], mx[r]);
                u64 e[NP];
#pragma unroll
                for (int p = 0; p < NP; ++p) {
                    float lo, hi;
                    unpack2(sub2(acc[r][p], mm), lo, hi);
                    e[p] = pack2(ex2_fast(lo), ex2_fast(hi));
                }
                es[r] = add2(e[0], e[1]);
#pragma unroll
                for (int p = 2; p < NP; p += 2) es[r] = add2(es[r], add2(e[p], e[p + 1]));
                float s0, s1;
                unpack2(es[r], s0, s1);
                grow = grow || !(s0 + s1 <= 1024.f);
            }
            if (grow) {                                        // rare: lazy rescale, terms stay below 2^10
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float a[CW];
#pragma unroll
                    for (int p = 0; p < NP; ++p) unpack2(acc[r][p], a[2 * p], a[2 * p + 1]);
                    float mt = fmaxf(a[0], a[1]);
#pragma unroll
                    for (int e = 2; e < CW; ++e) mt = fmaxf(mt, a[e]);
                    // the row's OWN sum decides (not a sibling row's that happened to trip the branch): a
                    // row's bits must not depend on which rows share its thread
                    float q0, q1;
                    unpack2(es[r], q0, q1);
                    if (!(q0 + q1 <= 1024.f)) {
                        const float mn = ceilf(mt);
                        const float fac = pow2i(mx[r] - mn);
                        float t0, t1;
                        unpack2(ts[r], t0, t1);
                        ts[r] = pack2(t0 * fac, t1 * fac);
                        sd[r] *= (double)fac;
                        mx[r] = mn;
                        float q = 0.f;
#pragma unroll
                        for (int e = 0; e < CW; ++e) q += ex2_fast(a[e] - mn);
                        es[r] = pack2(q, 0.f);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < R; ++r) ts[r] = add2(ts[r], es[r]);
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float t0, t1;
            unpack2(ts[r], t0, t1);
            sd[r] += (double)(t0 + t1);
            ts[r] = 0ull;
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ float64 arguments
// XF = 1: exponentials on the fp32 special-function unit; XF = 0: software exp2 in float64.
template <int DP, int CS, int XF, int R>
__device__ __forceinline__ void stream_f64(double *sm, const double *colc, const double *colt,
                                           const int cp, const int ncols,
                                           const double (&xr)[R][DP],
                                           const int tid, const int cs,
                                           const double (&est)[R],
                                           float (&mx)[R], double (&sd)[R])
{
    constexpr int CW = Tune<double, DP>::CW;
    constexpr int TJ = TileCols<double, DP, CS>::value;
    constexpr int STEPS = TJ / (CW * CS);
    constexpr int NR = DP + 1;
    constexpr int STAGE = (DP + 2) * TJ;

    float ts[R];
    double md[R];
    const int ntiles = (ncols + TJ - 1) / TJ;
    load_tile<double, DP, TJ, NR>(sm, colc, colt, colt, cp, 0, tid);
    cp_async_commit();
    // the reference points only now: the loads behind `est` have been in flight beside the tile's
#pragma unroll
    for (int r = 0; r < R; ++r) {
        mx[r] = (fabs(est[r]) < 1.0e7) ? ceilf((float)est[r]) : NEG_BIG;
        md[r] = (double)mx[r]; ts[r] = 0.f; sd[r] = 0.0;
    }
    for (int t = 0; t < ntiles; ++t) {
        if (t + 1 < ntiles) {
            load_tile<double, DP, TJ, NR>(sm + ((t + 1) & 1) * STAGE, colc, colt, colt, cp, (t + 1) * TJ, tid);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const double *st = sm + (t & 1) * STAGE;
#pragma unroll 1
        for (int q = 0; q < STEPS; ++q) {
            const int jj = (q * CS + cs) * CW;
            double acc[R][CW];
#pragma unroll
            for (int h = 0; h < CW / 2; ++h) {
                const double2 c0 = *reinterpret_cast<const double2 *>(st + DP * TJ + jj + 2 * h);
#pragma unroll
                for (int r = 0; r < R; ++r) { acc[r][2 * h] = c0.x; acc[r][2 * h + 1] = c0.y; }
            }
#pragma unroll
            for (int k = 0; k < DP; ++k) {
#pragma unroll
                for (int h = 0; h < CW / 2; ++h) {
                    const double2 y0 = *reinterpret_cast<const double2 *>(st + k * TJ + jj + 2 * h);
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        acc[r][2 * h] = fma(xr[r][k], y0.x, acc[r][2 * h]);
                        acc[r][2 * h + 1] = fma(xr[r][k], y0.y, acc[r][2 * h + 1]);
                    }
                }
            }
            if (XF) {
                // shifted arguments in fp32, their exponentials against the reference as it stands;
                // only a step whose sum exceeds 2^10 (or is not finite) moves the reference
                float v[R][CW], e2[R];
                bool grow = false;
#pragma unroll
                for (int r = 0; r < R; ++r) {
#pragma unroll
                    for (int e = 0; e < CW; ++e) v[r][e] = (float)(acc[r][e] - md[r]);
                    e2[r] = 0.f;
#pragma unroll
                    for (int e = 0; e < CW; ++e) e2[r] += ex2_fast(v[r][e]);
                    grow = grow || !(e2[r] <= 1024.f);
                }
                if (grow) {                                   // rare: move the reference point up
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        double mt = acc[r][0];
#pragma unroll
                        for (int e = 1; e < CW; ++e) mt = fmax(mt, acc[r][e]);
                        if (!(e2[r] <= 1024.f)) {                         // the row's own sum decides, never a sibling's
                            const float mn = ceilf((float)mt) + 1.0f;      // +1: the fp32 copy may round down
                            const float fac = pow2i(mx[r] - mn);
                            ts[r] *= fac;
                            sd[r] *= (double)fac;
                            mx[r] = mn;
                            md[r] = (double)mn;
                            e2[r] = 0.f;
#pragma unroll
                            for (int e = 0; e < CW; ++e) e2[r] += ex2_fast((float)(acc[r][e] - md[r]));
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < R; ++r) ts[r] += e2[r];
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    double mt = acc[r][0];
#pragma unroll
                    for (int e = 1; e < CW; ++e) mt = fmax(mt, acc[r][e]);
                    if (mt > md[r] + 8.0) {
                        const float mn = ceilf((float)mt) + 1.0f;
                        sd[r] *= (double)pow2i(mx[r] - mn);
                        mx[r] = mn;
                        md[r] = (double)mn;
                    }
#pragma unroll
                    for (int e = 0; e < CW; ++e) sd[r] += exp2(acc[r][e] - md[r]);
                }
            }
        }
        if (XF) {
#pragma unroll
            for (int r = 0; r < R; ++r) { sd[r] += (double)ts[r]; ts[r] = 0.f; }
        }
        __syncthreads();
    }
}

// Float64 epilogue of ONE row of a leg: `m` is the integer-valued maximum and `s` the sum of
// 2^(arg - m) over ALL columns, `h` the fp32 shift a difference-form row carried.  Writes the
// updated potential (unless the leg only checks, or the lane is frozen) and returns the row's
// term of the marginal residual (zero for the g-leg, which measures nothing).
template <typename T>
__device__ __forceinline__ double finish_one_row(const Dev &P, const Ctl &c, const int leg, const int slot, const int form,
                                                 const int i, const float m, const double s, const float h, const bool writes)
{
    const bool rows_x = (leg == LEG_F);
    const int rp = rows_x ? P.np : P.mp;
    const double *prow = (rows_x ? P.phi[c.parity] : P.gam) + (size_t)slot * rp;
    const size_t o = (size_t)slot * rp + i;
    const double lw = (rows_x ? P.la2 : P.lb2)[o];
    const double sq = (rows_x ? P.sqx : P.sqy)[o];
    const double pold = prow[i];
    const double L = (double)m + log2(s);
    // log2 of this row's marginal under the potentials the leg started from, and the
    // updated potential that makes the marginal equal to the weight (Eq. 3)
    double lmarg, pnew;
    if (form == FORM_DOT) {
        pnew = lw + sq - L;
        lmarg = lw + pold - pnew;
    } else {
        lmarg = L - ((double)h - pold);
        pnew = pold + (lw - lmarg);
    }
    double term = 0.0;
    if (leg != LEG_G) term = (rows_x ? P.wa : P.wb)[o] * fabs(expm1((lmarg - lw) * 0.6931471805599453));
    if (writes) {
        T hi, lo;
        if (form == FORM_DOT) { hi = (T)(pnew - sq); lo = T(0); }
        else { hi = (T)pnew; lo = (T)(pnew - (double)hi); }
        if (leg == LEG_F) {
            P.phi[c.parity ^ 1][o] = pnew;
            reinterpret_cast<T *>(P.ft[c.parity ^ 1])[o] = hi;
            reinterpret_cast<T *>(P.fl[c.parity ^ 1])[o] = lo;
        } else {
            P.gam[o] = pnew;
            reinterpret_cast<T *>(P.gt)[o] = hi;
            reinterpret_cast<T *>(P.gl)[o] = lo;
        }
    }
    return term;
}

// A row's term of the marginal residual in fixed point.  Terms are summed as integers from here
// on (registers, shuffles, shared memory, one atomic per row block on the lane's total), so the
// total is exact and does not depend on how rows are grouped into threads and blocks nor on
// the order in which blocks arrive.  A term that is not finite marks the lane instead.
__device__ __forceinline__ unsigned long long residual_fixed(const Dev &P, const int leg, const int slot,
                                                             const double term, const bool frozen)
{
    if (!isfinite(term)) {
        if (leg != LEG_F || !frozen) P.nonfinite[slot] = 1;
        return 0ull;
    }
    return __double2ull_rn(fmin(term, RSUM_ROW_MAX) * RSUM_SCALE);
}
__device__ __forceinline__ void finish_lane_residual(const Dev &P, const int leg, const int slot, const unsigned long long block_sum)
{
    atomicAdd((leg == LEG_F ? P.rsum_row : P.rsum_col) + slot, block_sum);
}

// Float64 epilogue of a CTA's RB rows (one thread per row) and the fused residual reduction.
// row_m / row_s hold, per CTA-local row, the integer-valued maximum and the sum of
// 2^(arg - max) over ALL columns; row_h the fp32 shift a difference-form row carried.
template <typename T, int RB, int THREADS = UPD_THREADS>
__device__ __forceinline__ void finish_rows(const Dev &P, const Ctl &c, const int leg, const int slot,
                                            const int form, const float *row_m, const double *row_s,
                                            const float *row_h, double *red)
{
    constexpr int NWARP = THREADS / 32;
    const int nrows = (leg == LEG_F) ? P.n : P.m;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool frozen = (P.mode == MODE_MASKED) && P.state[slot] != 0;
    const bool writes = !frozen && leg != LEG_V && !P.dry_run;
    unsigned long long term_sum = 0ull;
    for (int lr = tid; lr < RB; lr += THREADS) {
        const int i = blockIdx.x * RB + lr;
        if (i >= nrows) continue;
        const double term = finish_one_row<T>(P, c, leg, slot, form, i, row_m[lr], row_s[lr], row_h[lr], writes);
        if (leg != LEG_G) term_sum += residual_fixed(P, leg, slot, term, frozen);
    }
    if (leg == LEG_G || P.dry_run) return;

    // fused marginal-residual reduction -> one exact total per lane
    unsigned long long *redu = reinterpret_cast<unsigned long long *>(red);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) term_sum += __shfl_down_sync(0xffffffffu, term_sum, off);
    if (lane == 0) redu[warp] = term_sum;
    __syncthreads();
    if (tid == 0) {
        unsigned long long s = 0ull;
#pragma unroll
        for (int w = 0; w < NWARP; ++w) s += redu[w];
        finish_lane_residual(P, leg, slot, s);
    }
}

// Shared-memory scratch of one leg besides the column tiles.
template <int RB>
struct LegScratch {
    double row_s[RB];
    float row_m[RB];
    float row_h[RB];
    double red[UPD_THREADS / 32];
};

// One leg for the row block blockIdx.x of the lane in `slot`: row operands, streaming reduction over
// all columns, float64 epilogue, residual terms.  `c` supplies the cycle count and the buffer parity
// of the state the leg starts from.  PDL_EARLY: this is an f-leg launched as a kernel of its own,
// which reads its row operands while the kernel before it is still finishing and waits for it only
// before the column terms.  A row's arithmetic does not depend on the thread that holds it, nor on
// whether the leg runs as its own launch or inside the multi-cycle kernel below, so every way of
// running it gives the same bits.
template <typename T, int DP, int CS, int XF, int R, bool PDL_EARLY>
__device__ __forceinline__ void run_leg(const Dev &P, const Ctl &c, const int leg, const int slot, T *sm,
                                        LegScratch<(UPD_THREADS / 32) * R * (32 / CS)> &sc)
{
    constexpr int RG = 32 / CS;                  // row groups per warp
    constexpr int RW = R * RG;                   // rows per warp
    constexpr int NWARP = UPD_THREADS / 32;
    constexpr int RB = NWARP * RW;               // rows per CTA

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
    // lanes that share a row's columns sit RG apart, so that each quarter-warp reads a single
    // shared-memory address per load when CS <= 4 (a broadcast, the cheapest access pattern)
    const int cs = lane / RG, rg = lane % RG;
    const int lrow0 = warp * RW + rg * R;                // this thread's R consecutive CTA-local rows
    const int row0 = blockIdx.x * RB + lrow0;

    // the float64 epilogue's operands (one thread per row, much later): start them on their way to
    // L1 now, so that the epilogue does not begin with a round trip to L2 (the column tiles
    // stream through cp.async and leave L1 alone)
    for (int lr = tid; lr < RB; lr += UPD_THREADS) {
        const int i = blockIdx.x * RB + lr;
        if (i < nrows) {
            const size_t o = (size_t)slot * rp + i;
            asm volatile("prefetch.global.L1 [%0];" ::"l"((rows_x ? P.la2 : P.lb2) + o));
            asm volatile("prefetch.global.L1 [%0];" ::"l"((rows_x ? P.sqx : P.sqy) + o));
            asm volatile("prefetch.global.L1 [%0];" ::"l"(prow + i));
            if (leg != LEG_G) asm volatile("prefetch.global.L1 [%0];" ::"l"((rows_x ? P.wa : P.wb) + o));
        }
    }

    // R consecutive rows of one dimension are one aligned vector load (padding rows hold zeros)
    T xr[R][DP];
    T ph[R];
#pragma unroll
    for (int k = 0; k < DP; ++k) {
        T v[R];
        load_rows<T, R>(rowc + (size_t)k * rp + row0, row0 < rp, v);
#pragma unroll
        for (int r = 0; r < R; ++r) xr[r][k] = v[r];
    }
#pragma unroll
    for (int r = 0; r < R; ++r) ph[r] = (row0 + r < nrows && form == FORM_DIFF) ? (T)prow[row0 + r] : T(0);

    if (PDL_EARLY && leg == LEG_F) asm volatile("griddepcontrol.wait;" ::: "memory");

    float mx[R];
    double sd[R];
    // Where the exponential runs in fp32 on float64 arguments, the reference point of each row
    // starts at the value its log-sum-exp takes if the potential does not move in this leg
    // (Eq. 3 solved for the sum: L = log2 w + s|x|^2 - phi_old).  Near convergence that is within
    // a fraction of a unit of the truth, so the rescale branch of the streaming loop stays cold.
    // A reference far too HIGH would push every term towards the flush-to-zero range: such a CTA
    // repeats the pass from "minus infinity", as the other arithmetic modes always do.
    double m0[R];                                        // |m0| >= 1e7 stands for "no estimate"
#pragma unroll
    for (int r = 0; r < R; ++r) m0[r] = (double)NEG_BIG;
    if constexpr (sizeof(T) == 8 && XF != 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (row0 + r < nrows) {
                const size_t o = (size_t)slot * rp + row0 + r;
                m0[r] = (rows_x ? P.la2 : P.lb2)[o] + (rows_x ? P.sqx : P.sqy)[o] - prow[row0 + r];
            }
        }
    }
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        if constexpr (sizeof(T) == 4) {
            if (form == FORM_DOT) stream_f32<DP, CS, FORM_DOT, R>(sm, colc, colt, coll, cp, ncols, xr, ph, tid, cs, mx, sd);
            else stream_f32<DP, CS, FORM_DIFF, R>(sm, colc, colt, coll, cp, ncols, xr, ph, tid, cs, mx, sd);
        } else {
            stream_f64<DP, CS, XF, R>(sm, colc, colt, cp, ncols, xr, tid, cs, m0, mx, sd);
        }

        // merge the CS column splits of each row: maxima are integers, so the scalings are exact
#pragma unroll
        for (int off = 1; off < CS; off <<= 1) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float mo = __shfl_xor_sync(0xffffffffu, mx[r], off * RG);
                const double so = __shfl_xor_sync(0xffffffffu, sd[r], off * RG);
                const float mn = fmaxf(mx[r], mo);
                sd[r] = sd[r] * (double)pow2i(mx[r] - mn) + so * (double)pow2i(mo - mn);
                mx[r] = mn;
            }
        }
        if constexpr (sizeof(T) == 8 && XF != 0) {
            if (pass == 0) {
                bool low = false;
#pragma unroll
                for (int r = 0; r < R; ++r)
                    low = low || (row0 + r < nrows && fabs(m0[r]) < 1.0e7 && !(sd[r] >= 0x1p-20));
                if (!__syncthreads_or(low ? 1 : 0)) break;
                // only the rows whose estimate failed start over from "minus infinity"; the others
                // repeat the very same pass (same bits), so that a row's result does not depend on
                // which rows share its block
#pragma unroll
                for (int r = 0; r < R; ++r)
                    if (row0 + r < nrows && fabs(m0[r]) < 1.0e7 && !(sd[r] >= 0x1p-20)) m0[r] = (double)NEG_BIG;
                continue;
            }
        }
        break;
    }
    if (cs == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            sc.row_m[lrow0 + r] = mx[r];
            sc.row_s[lrow0 + r] = sd[r];
            sc.row_h[lrow0 + r] = (float)ph[r];
        }
    }
    __syncthreads();
    finish_rows<T, RB>(P, c, leg, slot, form, sc.row_m, sc.row_s, sc.row_h, sc.red);
}

// RR: rows per thread, 0 = the type's default.  Rows are independent and a row's arithmetic does
// not depend on which thread holds it, so launches with different RR give the same bits.
template <typename T, int DP, int CS, int XF, int RR = 0>
__global__ void __launch_bounds__(UPD_THREADS) update_kernel(const Dev P, const int leg)
{
    constexpr int R = RR ? RR : Tune<T, DP>::R;
    constexpr int RB = (UPD_THREADS / 32) * R * (32 / CS);   // rows per CTA

    extern __shared__ __align__(16) unsigned char smem_raw[];
    T *sm = reinterpret_cast<T *>(smem_raw);
    __shared__ LegScratch<RB> sc;

    // Programmatic dependent launch.  The f-leg follows the g-leg, which writes neither the control
    // block nor coordinates nor the row potentials: its control block, row coordinates and epilogue
    // operands are read while that g-leg is still finishing, and only the column terms wait.  The
    // other legs wait first; the g-leg releases its dependent (the next f-leg) only AFTER its own
    // wait, so that an early f-leg can rely on the planner and the move being complete.
    // (The column check also reads the control block early, then waits for the f-leg's verdict.)
    const bool early = (leg == LEG_F);
    if (leg == LEG_G) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const Ctl c = *P.ctl;
    if (leg == LEG_V) asm volatile("griddepcontrol.wait;" ::: "memory");
    const int slot = blockIdx.y;
    const bool idle = c.done || slot >= c.n_phys
                      || (P.early_exit && P.state[slot] != 0)   // early-exit mask arm: a frozen lane costs a launch slot only
                      || (leg != LEG_V && c.static_final)
                      || (leg == LEG_V && !(c.static_final || lane_flag(P, c, slot)))
                      || (int)blockIdx.x * RB >= (leg == LEG_F ? P.n : P.m);
    if (idle) {
        // Every kernel of the chain must wait at least once before it completes: a kernel's wait
        // covers its immediate predecessor only, and "everything earlier in the stream has finished"
        // follows from it only if that predecessor waited too.  An f-leg with nothing to do has not
        // waited yet, so its first block does so here (a batch that is finished, or another batch's
        // kernels in the same stream, would otherwise let later kernels overtake a running g-leg).
        if (early && blockIdx.x == 0 && blockIdx.y == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    run_leg<T, DP, CS, XF, R, true>(P, c, leg, slot, sm, sc);
}

// ------------------------------------------------------------------ several cycles per launch
// One thread-block CLUSTER per lane: block r of the cluster owns row block r of both clouds and the
// cluster walks the lane through up to `cycles` whole cycles inside one launch -
//     f-leg (with the row screen of the state before it) -> [column check if screen-positive] ->
//     verdict -> retire, or g-leg and on to the next cycle
// - so that a cycle costs two or three cluster barriers instead of a chain of five dependent
// launches.  Lanes are independent problems (Eq. 2): clusters never wait for one another, and
// inside a cluster the only synchronisation is the hardware cluster barrier, which every thread of
// every block reaches on every path (all blocks of a cluster take the same decisions from the same
// values).  Blocks hand the potentials to one another through global memory (the column terms are
// read by cp.async, which bypasses L1, after the barrier's release/acquire).
// A lane that passes the two-sided check (Eq. 5) writes its own outputs and leaves; the planner that
// follows the launch does the accounting of Eq. 6-8 for all cycles of the launch at once and fills
// the holes (Section "Screen, verify, and compact").  The legs are run_leg, so the bits are those
// of the one-launch-per-leg path.
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned long long ld_cg_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.global.cg.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_cg_s32(const int *p)
{
    int v;
    asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

template <typename T, int DP, int CS, int XF, int RR = 0>
__global__ void __launch_bounds__(UPD_THREADS) lane_cycles_kernel(const Dev P, const int cycles)
{
    constexpr int R = RR ? RR : Tune<T, DP>::R;
    constexpr int RB = (UPD_THREADS / 32) * R * (32 / CS);

    extern __shared__ __align__(16) unsigned char smem_raw[];
    T *sm = reinterpret_cast<T *>(smem_raw);
    __shared__ LegScratch<RB> sc;

    pdl_enter();
    Ctl c = *P.ctl;                              // private copy: cycle and parity advance per lane below
    const int slot = blockIdx.y;
    if (c.done || slot >= c.n_phys) return;      // the whole cluster takes this exit together
    const int tid = threadIdx.x;
    const int lane_id = P.lane_id[slot];
    const double inv_s = 1.0 / P.scale[slot];
    unsigned long long seen_row = 0ull, seen_col = 0ull;     // totals already accounted for (the sums are only cleared at the end)
    int checks = 0, retired_at = 0;

    for (int it = 0; it < cycles; ++it) {
        // f-leg of cycle k+1; its epilogue also yields the row residual of the state after k cycles
        run_leg<T, DP, CS, XF, R, false>(P, c, LEG_F, slot, sm, sc);
        cluster_sync_all();
        const unsigned long long tot_row = ld_cg_u64(P.rsum_row + slot);
        const double rr = (double)(tot_row - seen_row) * (1.0 / RSUM_SCALE);
        seen_row = tot_row;
        int nf = ld_cg_s32(P.nonfinite + slot);
        const int k = c.cycle;
        const bool audited = (k >= 1 && (k % P.audit_every) == 0) || (k == 0 && P.audit_initial);
        const bool fl = audited && !nf && rr <= P.tol_screen;
        double rc = 0.0;
        if (fl) {                                // two-sided check: the column marginal, genuinely measured
            run_leg<T, DP, CS, XF, R, false>(P, c, LEG_V, slot, sm, sc);
            cluster_sync_all();
            const unsigned long long tot_col = ld_cg_u64(P.rsum_col + slot);
            rc = (double)(tot_col - seen_col) * (1.0 / RSUM_SCALE);
            seen_col = tot_col;
            nf = ld_cg_s32(P.nonfinite + slot);
            ++checks;
        }
        const bool vd = !nf && fmax(rr, rc) <= P.tol_stop;
        const bool limit = k >= P.max_iter;
        int st = LANE_RUNNING;
        if (nf) st = LANE_NONFINITE;
        else if (fl && vd) st = LANE_DONE;
        else if (limit) st = LANE_ITER_LIMIT;
        if (st != LANE_RUNNING) {
            // retire: this block's rows of the potentials of the audited state, in the caller's units
            const double *phi = P.phi[c.parity] + (size_t)slot * P.np;
            const double *gam = P.gam + (size_t)slot * P.mp;
            for (int lr = tid; lr < RB; lr += UPD_THREADS) {
                const int i = blockIdx.x * RB + lr;
                if (i < P.n) P.f_out[(size_t)lane_id * P.n + i] = phi[i] * inv_s;
                if (i < P.m) P.g_out[(size_t)lane_id * P.m + i] = gam[i] * inv_s;
            }
            if (blockIdx.x == 0 && tid == 0) {
                P.res_row[lane_id] = rr;
                P.res_col[lane_id] = fl ? rc : __longlong_as_double(0x7ff8000000000000LL);
                P.depth[lane_id] = (limit && st != LANE_DONE) ? P.max_iter : k;
                P.status[lane_id] = st;
                P.emitted[lane_id] = 1;
            }
            retired_at = k + 1;
            break;
        }
        c.cycle = k + 1;
        c.parity ^= 1;
        run_leg<T, DP, CS, XF, R, false>(P, c, LEG_G, slot, sm, sc);
        cluster_sync_all();
    }
    // hand over to the planner: when the lane left (0 = still running) and how many column checks
    // it ran.  The residual sums are left as they are (another block of the cluster may still be
    // reading them); the planner clears them.
    if (blockIdx.x == 0 && tid == 0) {
        P.ret_at[slot] = retired_at;
        P.n_checks[slot] = checks;
    }
}

}  // namespace skb
