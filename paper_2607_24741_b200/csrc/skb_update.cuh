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
// (fp32, d <= 4: two rows measured faster than four at every width of the registration workload -
// f-leg 609 against 628 us at 32 lanes, 319 against 331 us at 16 - because twice the blocks balance
// better over the SMs, which outweighs the extra shared-memory loads per pair.)
template <int DP> struct Tune<float, DP> {
    static constexpr int R = DP <= 4 ? 2 : (DP <= 8 ? 4 : (DP == 16 ? SKB_F32_R16 : 2));
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
// RES = 1: every column tile of the lane is already resident in shared memory (tile t at
// sm + t * res_stride, its term rows at row res_trow and res_trow + 1 of the tile); nothing is
// loaded and no block-wide barrier is needed.  Same steps in the same order, same bits.
template <int DP, int CS, int FORM, int R, int RES = 0>
__device__ __forceinline__ void stream_f32(float *sm, const float *colc, const float *colt, const float *coll,
                                           const int cp, const int ncols,
                                           const float (&xrow)[R][DP],
                                           const float (&ph)[R], const int tid, const int cs,
                                           float (&mx)[R], double (&sd)[R],
                                           const int res_stride = 0, const int res_trow = 0)
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
    const int ctoff = RES ? res_trow * TJ : DP * TJ, cloff = ctoff + TJ;
    if constexpr (!RES) {
        load_tile<float, DP, TJ, NR>(sm, colc, colt, coll, cp, 0, tid);
        cp_async_commit();
    }
    for (int t = 0; t < ntiles; ++t) {
        if constexpr (!RES) {
            if (t + 1 < ntiles) {
                load_tile<float, DP, TJ, NR>(sm + ((t + 1) & 1) * STAGE, colc, colt, coll, cp, (t + 1) * TJ, tid);
                cp_async_commit();
                cp_async_wait<1>();
            } else {
                cp_async_wait<0>();
            }
            __syncthreads();
        }
        const float *st = RES ? sm + t * res_stride : sm + (t & 1) * STAGE;
        constexpr int UQ = SKB_UNROLL_Q;
#pragma unroll UQ
        for (int q = 0; q < STEPS; ++q) {
            const int jj = (q * CS + cs) * CW;
            u64 acc[R][NP];
            u64 ct[NP];
#pragma unroll
            for (int h = 0; h < NP / 2; ++h) {
                const ulonglong2 c = *reinterpret_cast<const ulonglong2 *>(st + ctoff + jj + 4 * h);
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
                    const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(st + cloff + jj + 4 * h);
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
        if constexpr (!RES) __syncthreads();
    }
}

// ------------------------------------------------------------------ float64 arguments
// XF = 1: exponentials on the fp32 special-function unit; XF = 0: software exp2 in float64.
template <int DP, int CS, int XF, int R, int RES = 0>
__device__ __forceinline__ void stream_f64(double *sm, const double *colc, const double *colt,
                                           const int cp, const int ncols,
                                           const double (&xr)[R][DP],
                                           const int tid, const int cs,
                                           const double (&est)[R],
                                           float (&mx)[R], double (&sd)[R],
                                           const int res_stride = 0, const int res_trow = 0)
{
    constexpr int CW = Tune<double, DP>::CW;
    constexpr int TJ = TileCols<double, DP, CS>::value;
    constexpr int STEPS = TJ / (CW * CS);
    constexpr int NR = DP + 1;
    constexpr int STAGE = (DP + 2) * TJ;

    float ts[R];
    double md[R];
    const int ntiles = (ncols + TJ - 1) / TJ;
    const int ctoff = RES ? res_trow * TJ : DP * TJ;
    if constexpr (!RES) {
        load_tile<double, DP, TJ, NR>(sm, colc, colt, colt, cp, 0, tid);
        cp_async_commit();
    }
    // the reference points only now: the loads behind `est` have been in flight beside the tile's
#pragma unroll
    for (int r = 0; r < R; ++r) {
        mx[r] = (fabs(est[r]) < 1.0e7) ? ceilf((float)est[r]) : NEG_BIG;
        md[r] = (double)mx[r]; ts[r] = 0.f; sd[r] = 0.0;
    }
    for (int t = 0; t < ntiles; ++t) {
        if constexpr (!RES) {
            if (t + 1 < ntiles) {
                load_tile<double, DP, TJ, NR>(sm + ((t + 1) & 1) * STAGE, colc, colt, colt, cp, (t + 1) * TJ, tid);
                cp_async_commit();
                cp_async_wait<1>();
            } else {
                cp_async_wait<0>();
            }
            __syncthreads();
        }
        const double *st = RES ? sm + t * res_stride : sm + (t & 1) * STAGE;
#pragma unroll 1
        for (int q = 0; q < STEPS; ++q) {
            const int jj = (q * CS + cs) * CW;
            double acc[R][CW];
#pragma unroll
            for (int h = 0; h < CW / 2; ++h) {
                const double2 c0 = *reinterpret_cast<const double2 *>(st + ctoff + jj + 2 * h);
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
        if constexpr (!RES) __syncthreads();
    }
}

// The arithmetic of one row's epilogue.  m: integer-valued maximum, s: sum of 2^(arg - m) over all
// columns, h: the fp32 shift a difference-form row carried, pold: the potential the leg started
// from.  Gives the updated potential that makes the row's marginal equal to its weight (Eq. 3) and,
// where asked, the row's term w |marginal/weight - 1| of the L1 residual of the state before the leg.
__device__ __forceinline__ void row_math(const int form, const bool want_term, const double lw, const double sq,
                                         const double w, const double pold, const float m, const double s,
                                         const float h, double &pnew, double &term)
{
    const double L = (double)m + log2(s);
    double lmarg;                          // log2 of the row's marginal under the potentials the leg started from
    if (form == FORM_DOT) {
        pnew = lw + sq - L;
        lmarg = lw + pold - pnew;
    } else {
        lmarg = L - ((double)h - pold);
        pnew = pold + (lw - lmarg);
    }
    term = want_term ? w * fabs(expm1((lmarg - lw) * 0.6931471805599453)) : 0.0;
}
// The per-point term the opposite leg streams: high part (expanded form: potential minus the scaled
// squared norm) and low part (difference form only).
template <typename T>
__device__ __forceinline__ void split_potential(const int form, const double pnew, const double sq, T &hi, T &lo)
{
    if (form == FORM_DOT) { hi = (T)(pnew - sq); lo = T(0); }
    else { hi = (T)pnew; lo = (T)(pnew - (double)hi); }
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
    double pnew, term;
    row_math(form, leg != LEG_G, lw, sq, leg != LEG_G ? (rows_x ? P.wa : P.wb)[o] : 0.0, pold, m, s, h, pnew, term);
    if (writes) {
        T hi, lo;
        split_potential<T>(form, pnew, sq, hi, lo);
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
                                            const float *row_h, double *red, const int row_base)
{
    constexpr int NWARP = THREADS / 32;
    const int nrows = (leg == LEG_F) ? P.n : P.m;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool frozen = (P.mode == MODE_MASKED) && P.state[slot] != 0;
    const bool writes = !frozen && leg != LEG_V && !P.dry_run;
    unsigned long long term_sum = 0ull;
    for (int lr = tid; lr < RB; lr += THREADS) {
        const int i = row_base + lr;
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

// Merge of the CS column splits of each row (lanes RG = 32 / CS apart hold the same rows): maxima are
// integers, so the scalings are exact powers of two and each sum is rounded once.
template <int CS, int R>
__device__ __forceinline__ void merge_splits(float (&mx)[R], double (&sd)[R])
{
    constexpr int RG = 32 / CS;
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
}

// Shared-memory scratch of one leg besides the column tiles.
template <int RB>
struct LegScratch {
    double row_s[RB];
    float row_m[RB];
    float row_h[RB];
    double red[UPD_THREADS / 32];
};

// One leg for the RB rows from `row_base` on of the lane in `slot`: row operands, streaming reduction over
// all columns, float64 epilogue, residual terms.  `c` supplies the cycle count and the buffer parity
// of the state the leg starts from.  PDL_EARLY: this is an f-leg launched as a kernel of its own,
// which reads its row operands while the kernel before it is still finishing and waits for it only
// before the column terms.  A row's arithmetic does not depend on the thread that holds it, nor on
// whether the leg runs as its own launch or inside the multi-cycle kernel below, so every way of
// running it gives the same bits.
template <typename T, int DP, int CS, int XF, int R, bool PDL_EARLY, int RBS = (UPD_THREADS / 32) * R * (32 / CS)>
__device__ __forceinline__ void run_leg(const Dev &P, const Ctl &c, const int leg, const int slot, T *sm,
                                        LegScratch<RBS> &sc, const int row_base)
{
    static_assert(RBS >= (UPD_THREADS / 32) * R * (32 / CS), "scratch smaller than the row block");
    constexpr int RG = 32 / CS;                  // row groups per warp
    constexpr int RW = R * RG;                   // rows per warp
    constexpr int NWARP = UPD_THREADS / 32;
    constexpr int RB = NWARP * RW;               // rows per CTA

    // roles: rows are x-points for the f-leg, y-points otherwise
    const bool rows_x = (leg == LEG_F);
    const int nrows = rows_x ? P.n : P.m, rp = rows_x ? P.np : P.mp;
    const int ncols = rows_x ? P.m : P.n, cp = rows_x ? P.mp : P.np;
    if (row_base >= nrows) return;
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
    const int row0 = row_base + lrow0;

    // the float64 epilogue's operands (one thread per row, much later): start them on their way to
    // L1 now, so that the epilogue does not begin with a round trip to L2 (the column tiles
    // stream through cp.async and leave L1 alone)
    for (int lr = tid; lr < RB; lr += UPD_THREADS) {
        const int i = row_base + lr;
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

        merge_splits<CS, R>(mx, sd);
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
    finish_rows<T, RB>(P, c, leg, slot, form, sc.row_m, sc.row_s, sc.row_h, sc.red, row_base);
}

// Guard band on the one-launch-per-leg path: with it on, a column-check launch carries a pool of extra
// blocks (grid rows past the lanes).  The pool looks for lanes whose fused screen came out inside the
// band and re-evaluates their row residual from the raw inputs in float64 - one warp per row, all pool
// warps sharing a lane's rows, exact integer sum - and the planner decides from that value.
// (Its float64 exponentials need more registers than the fp32 legs: update_kernel's launch bounds keep
// the fp32 instances at four blocks per SM, and the surplus spills here, on the rare path.)
template <bool VEC = false>
__device__ __forceinline__ void guard_pool(const Dev &P, const Ctl &c, const int nlanes, unsigned long long *red)
{
    if (c.done || c.static_final) return;
    constexpr int NW = UPD_THREADS / 32;
    __shared__ int hot[UPD_THREADS];
    __shared__ int n_hot;
    const int pool_id = ((int)blockIdx.y - nlanes) * (int)gridDim.x + (int)blockIdx.x;
    const int pool_warps = ((int)gridDim.y - nlanes) * (int)gridDim.x * NW;
    for (int s0 = 0; s0 < c.n_phys; s0 += UPD_THREADS * 4) {
        if (threadIdx.x == 0) n_hot = 0;
        __syncthreads();
        // all loads first (independent, clamped to a valid slot), then the predicates: the scan is on the
        // launch's critical path and a short-circuit chain would pay one memory latency per term
        int st_[4], fr_[4], nf_[4];
        unsigned long long rs_[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int s = s0 + u * UPD_THREADS + (int)threadIdx.x;
            const int sl = s < c.n_phys ? s : 0;
            st_[u] = P.start[sl];
            fr_[u] = P.state[sl];
            nf_[u] = P.nonfinite[sl];
            rs_[u] = P.rsum_row[sl];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int s = s0 + u * UPD_THREADS + (int)threadIdx.x;
            if (s < c.n_phys && lane_audited(P, c.cycle, st_[u]) && !(P.mode != MODE_ACTIVE && fr_[u] != 0) &&
                !nf_[u] && in_guard_band(P, (double)rs_[u] * (1.0 / RSUM_SCALE))) {
                const int at = atomicAdd(&n_hot, 1);
                if (at < UPD_THREADS) hot[at] = s;
            }
        }
        __syncthreads();
        const int nh = n_hot < UPD_THREADS ? n_hot : UPD_THREADS;   // more than 128 at once: the rest keep their fp32 screen
        for (int q = 0; q < nh; ++q) {
            const int s = hot[q];
            int bad;
            const unsigned long long mine = direct_rows_block<NW, VEC>(P, s, pool_id * NW, pool_warps, P.n,
                                                                  P.phi[c.parity] + (size_t)s * P.np, 0, red, &bad);
            if (threadIdx.x == 0) {
                atomicAdd(P.rsum_row64 + s, mine);
                if (bad) P.nonfinite[s] = 1;
                P.esc[s] = 1;
            }
        }
        __syncthreads();
    }
}

// Blocks per SM the per-leg kernel is held to (register cap): four for fp32 up to 16 dimensions,
// five / three for float64 arguments with fp32 exponentials at two / four rows per thread - what the
// legs reach by themselves, so that the guard pool's float64 code, which lives in the same kernel,
// cannot cost them an occupancy step - and seven for fp32 up to 4 dimensions, where occupancy was
// measured to pay (registration f-leg at 32 / 8 lanes: 638 / - us at five blocks, 627 / 180 at six,
// 610 / 174 at seven, 614 / 190 at eight, 615 / 198 at ten).
#ifndef SKB_BLOCKS_F32_SMALL
#define SKB_BLOCKS_F32_SMALL 7
#endif
#ifndef SKB_BLOCKS_F32_MID
#define SKB_BLOCKS_F32_MID 4
#endif
#ifndef SKB_BLOCKS_F64_WIDE
#define SKB_BLOCKS_F64_WIDE 3
#endif
#ifndef SKB_BLOCKS_F64_NARROW
#define SKB_BLOCKS_F64_NARROW 5
#endif
template <typename T, int DP, int XF, int RR> struct UpdBlocksPerSM {
    static constexpr int R = RR ? RR : Tune<T, DP>::R;
    static constexpr int value = sizeof(T) == 4 ? (DP <= 4 ? SKB_BLOCKS_F32_SMALL : (DP <= 16 ? SKB_BLOCKS_F32_MID : 1))
                                                : ((DP <= 8 && XF == 1) ? (R >= 4 ? SKB_BLOCKS_F64_WIDE : SKB_BLOCKS_F64_NARROW) : 1);
};

// One leg as a launch of its own.  RR: rows per thread, 0 = the type's default.  Rows are independent
// and a row's arithmetic does not depend on which thread holds it, so launches with different RR
// give the same bits.
template <typename T, int DP, int CS, int XF, int RR = 0>
__global__ void __launch_bounds__(UPD_THREADS, UpdBlocksPerSM<T, DP, XF, RR>::value) update_kernel(const Dev P, const int leg, const int nlanes)
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
    const int row_base = (int)blockIdx.x * RB;
    if (leg == LEG_V && (int)blockIdx.y >= nlanes) {
        guard_pool(P, c, nlanes, reinterpret_cast<unsigned long long *>(sc.red));
        return;
    }
    const bool idle = c.done || slot >= c.n_phys
                      || (P.early_exit && P.state[slot] != 0)   // early-exit mask arm: a frozen lane costs a launch slot only
                      || (leg != LEG_V && c.static_final)
                      || (leg == LEG_V && !(c.static_final || lane_needs_column_check(P, c, slot)))
                      || row_base >= (leg == LEG_F ? P.n : P.m);
    if (idle) {
        // Every kernel of the chain must wait at least once before it completes: a kernel's wait
        // covers its immediate predecessor only, and "everything earlier in the stream has finished"
        // follows from it only if that predecessor waited too.  An f-leg with nothing to do has not
        // waited yet, so its first block does so here (a batch that is finished, or another batch's
        // kernels in the same stream, would otherwise let later kernels overtake a running g-leg).
        if (early && blockIdx.x == 0 && blockIdx.y == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    run_leg<T, DP, CS, XF, R, true>(P, c, leg, slot, sm, sc, row_base);
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

// Blocks per SM the multi-cycle kernels are held to.  The launch policy never asks for more than four
// blocks of them per SM, so up to 128 registers are free and the compiler is told so.  Deep float64
// variants keep the registers their streaming loops need.
template <typename T, int DP> struct LaneBlocksPerSM {
    static constexpr int value = DP <= 8 ? 4 : (DP == 16 ? 3 : (sizeof(T) == 4 ? 4 : 2));
};

template <typename T, int DP, int CS, int XF, int RR = 0>
__global__ void __launch_bounds__(UPD_THREADS, LaneBlocksPerSM<T, DP>::value) lane_cycles_kernel(const Dev P, const int cycles)
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
    const int start = P.start[slot];             // batch cycle at which this lane came in
    const double inv_s = 1.0 / P.scale[slot];
    unsigned long long seen_row = 0ull, seen_col = 0ull, seen_row64 = 0ull;     // totals already accounted for (the planner clears the sums)
    int checks = 0, retired_at = 0;

    // One call site for the three kinds of leg (the leg is a run-time value), so that the streaming
    // loops are instantiated once.  leg F: f-leg of cycle k+1, whose epilogue also yields the row
    // residual of the state after k cycles; leg V: column check of that state; leg G: g-leg.
    int leg = LEG_F, it = 0, nf = 0;
    double rr = 0.0, rc = 0.0;
    bool fl = false;
    for (;;) {
        run_leg<T, DP, CS, XF, R, false>(P, c, leg, slot, sm, sc, (int)blockIdx.x * RB);
        cluster_sync_all();
        if (leg == LEG_G) {
            if (++it >= cycles) break;
            leg = LEG_F;
            continue;
        }
        const int k = c.cycle;
        if (leg == LEG_F) {
            const unsigned long long tot_row = ld_cg_u64(P.rsum_row + slot);
            rr = (double)(tot_row - seen_row) * (1.0 / RSUM_SCALE);
            seen_row = tot_row;
            nf = ld_cg_s32(P.nonfinite + slot);
            const bool audited = lane_audited(P, k, start);
            if (audited && !nf && in_guard_band(P, rr)) {
                // guard band: decide from a float64 re-evaluation of the row residual
                int bad;
                const double *phi_lane = P.phi[c.parity] + (size_t)slot * P.np;
                const int r0 = (int)blockIdx.x * RB, r1 = min(r0 + RB, P.n);
                const unsigned long long mine = direct_rows_block<UPD_THREADS / 32>(
                    P, slot, r0, UPD_THREADS / 32, r1, phi_lane, 0, reinterpret_cast<unsigned long long *>(sc.red), &bad);
                if (tid == 0) {
                    atomicAdd(P.rsum_row64 + slot, mine);
                    if (bad) P.nonfinite[slot] = 1;
                }
                cluster_sync_all();
                const unsigned long long tot64 = ld_cg_u64(P.rsum_row64 + slot);
                rr = (double)(tot64 - seen_row64) * (1.0 / RSUM_SCALE);
                seen_row64 = tot64;
                nf = ld_cg_s32(P.nonfinite + slot);
            }
            fl = audited && !nf && rr <= P.tol_screen;
            rc = 0.0;
            if (fl) { leg = LEG_V; continue; }     // two-sided check: the column marginal, genuinely measured
        } else {
            const unsigned long long tot_col = ld_cg_u64(P.rsum_col + slot);
            rc = (double)(tot_col - seen_col) * (1.0 / RSUM_SCALE);
            seen_col = tot_col;
            nf = ld_cg_s32(P.nonfinite + slot);
            ++checks;
        }
        const bool vd = !nf && fmax(rr, rc) <= P.tol_stop;
        const bool limit = k - start >= P.max_iter;
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
                P.depth[lane_id] = (limit && st != LANE_DONE) ? P.max_iter : k - start;
                P.status[lane_id] = st;
                P.emitted[lane_id] = 1;
            }
            retired_at = k + 1;
            break;
        }
        c.cycle = k + 1;
        c.parity ^= 1;
        leg = LEG_G;
    }
    // hand over to the planner: when the lane left (0 = still running) and how many column checks
    // it ran.  The residual sums are left as they are (another block of the cluster may still be
    // reading them); the planner clears them.
    if (blockIdx.x == 0 && tid == 0) {
        P.ret_at[slot] = retired_at;
        P.n_checks[slot] = checks;
    }
}


// ------------------------------------------------------------------ several cycles per launch, lane in shared memory
// The same walk as lane_cycles_kernel, with the lane's whole state resident in the cluster's shared
// memory for the length of the launch: every block holds ALL column tiles of both clouds
// (coordinates and per-point terms, in the streaming kernels' tile layout) and the float64
// potentials and constants of its OWN rows.  A leg streams from shared memory; its epilogue
// writes each new per-point term into the tile copies of every block of the cluster (distributed
// shared memory) and the block's part of the residual into every block's table, and ONE cluster
// barrier per leg makes them visible.  Inside the loop nothing touches global memory but the
// (constant, L1-resident) row coordinates; the state is loaded once and written back once.
// Tile t of the y cloud: rows 0..DP-1 coordinates, row DP term, row DP+1 low part.
// Tile t of the x cloud: coordinates, then (term, low part) of buffer parity 0 and of parity 1: the
// f-leg writes the look-ahead potentials into the other parity while the column check may still
// need the current one.
template <typename V>
__device__ __forceinline__ void st_cluster(V *local, const unsigned rank, const V v)
{
    const unsigned laddr = (unsigned)__cvta_generic_to_shared(local);
    unsigned raddr;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(laddr), "r"(rank));
    if constexpr (sizeof(V) == 8) {
        unsigned long long bits;
        memcpy(&bits, &v, 8);
        asm volatile("st.shared::cluster.b64 [%0], %1;" ::"r"(raddr), "l"(bits) : "memory");
    } else {
        unsigned bits;
        memcpy(&bits, &v, 4);
        asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(raddr), "r"(bits) : "memory");
    }
}

template <typename T, int DP, int CS>
struct ResidentLayout {
    static constexpr int R = Tune<T, DP>::R;
    static constexpr int RB = (UPD_THREADS / 32) * R * (32 / CS);
    static constexpr int TJ = TileCols<T, DP, CS>::value;
    static constexpr int STY = (DP + 2) * TJ;
    static constexpr int STX = (DP + 4) * TJ;
    static constexpr int NDBL = 9;                     // float64 arrays of RB own rows each
    static size_t bytes(const int n, const int m)
    {
        const size_t ntx = (n + TJ - 1) / TJ, nty = (m + TJ - 1) / TJ;
        return sizeof(T) * (nty * STY + ntx * STX) + (size_t)NDBL * RB * sizeof(double);
    }
};

template <typename T, int DP, int CS, int XF>
__global__ void __launch_bounds__(UPD_THREADS, LaneBlocksPerSM<T, DP>::value) lane_resident_kernel(const Dev P, const int cycles)
{
    typedef ResidentLayout<T, DP, CS> L;
    constexpr int R = L::R, RB = L::RB, TJ = L::TJ, STY = L::STY, STX = L::STX;
    constexpr int RG = 32 / CS, RW = R * RG;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ LegScratch<RB> sc;
    __shared__ unsigned long long part[2][MAX_CLUSTER_RANKS];    // [row | column residual][block of the cluster]
    __shared__ int part_nf[2][MAX_CLUSTER_RANKS];

    pdl_enter();
    Ctl c = *P.ctl;
    const int slot = blockIdx.y;
    if (c.done || slot >= c.n_phys) return;      // the whole cluster takes this exit together
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x, NC = gridDim.x;
    const int ntY = (P.m + TJ - 1) / TJ, ntX = (P.n + TJ - 1) / TJ;
    T *colsY = reinterpret_cast<T *>(smem_raw);
    T *colsX = colsY + (size_t)ntY * STY;
    double *own = reinterpret_cast<double *>(colsX + (size_t)ntX * STX);
    double *lwx = own, *sqx = own + RB, *wax = own + 2 * RB, *lwy = own + 3 * RB, *sqy = own + 4 * RB, *wby = own + 5 * RB;
    double *potx[2] = {own + 6 * RB, own + 7 * RB};
    double *poty = own + 8 * RB;

    // ---- the lane comes in: all column tiles of both clouds, this block's rows of everything else
    const T *xs = reinterpret_cast<const T *>(P.xs) + (size_t)slot * DP * P.np;
    const T *ys = reinterpret_cast<const T *>(P.ys) + (size_t)slot * DP * P.mp;
    for (int t = 0; t < ntY; ++t)
        load_tile<T, DP, TJ, DP + 2>(colsY + (size_t)t * STY, ys, reinterpret_cast<const T *>(P.gt) + (size_t)slot * P.mp,
                                     reinterpret_cast<const T *>(P.gl) + (size_t)slot * P.mp, P.mp, t * TJ, tid);
    for (int t = 0; t < ntX; ++t) {
        load_tile<T, DP, TJ, DP + 2>(colsX + (size_t)t * STX, xs, reinterpret_cast<const T *>(P.ft[0]) + (size_t)slot * P.np,
                                     reinterpret_cast<const T *>(P.fl[0]) + (size_t)slot * P.np, P.np, t * TJ, tid);
        load_tile<T, 0, TJ, 2>(colsX + (size_t)t * STX + (DP + 2) * TJ, xs, reinterpret_cast<const T *>(P.ft[1]) + (size_t)slot * P.np,
                               reinterpret_cast<const T *>(P.fl[1]) + (size_t)slot * P.np, P.np, t * TJ, tid);
    }
    cp_async_commit();
    for (int lr = tid; lr < RB; lr += UPD_THREADS) {
        const int i = b * RB + lr;
        if (i < P.n) {
            const size_t o = (size_t)slot * P.np + i;
            lwx[lr] = P.la2[o]; sqx[lr] = P.sqx[o]; wax[lr] = P.wa[o];
            potx[0][lr] = P.phi[0][o]; potx[1][lr] = P.phi[1][o];
        }
        if (i < P.m) {
            const size_t o = (size_t)slot * P.mp + i;
            lwy[lr] = P.lb2[o]; sqy[lr] = P.sqy[o]; wby[lr] = P.wb[o];
            poty[lr] = P.gam[o];
        }
    }
    cp_async_wait<0>();
    const int form = (sizeof(T) == 8) ? (int)FORM_DOT : P.form[slot];
    const int lane_id = P.lane_id[slot];
    const int start = P.start[slot];             // batch cycle at which this lane came in
    const double inv_s = 1.0 / P.scale[slot];
    cluster_sync_all();                          // every block's tables exist before anyone writes into them

    // one leg on the resident state; leaves this block's part of the residual in every block's table
    auto leg_resident = [&](const int leg, const int parity) {
        const bool rows_x = (leg == LEG_F);
        const int nrows = rows_x ? P.n : P.m, rp = rows_x ? P.np : P.mp;
        const int ncols = rows_x ? P.m : P.n, cp = rows_x ? P.mp : P.np;
        unsigned long long block_sum = 0ull;
        int block_nf = 0;
        if (b * RB < nrows) {
            const T *rowc = rows_x ? xs : ys;
            T *cols = rows_x ? colsY : colsX;
            const int stride = rows_x ? STY : STX;
            const int trow = rows_x ? DP : DP + 2 * parity;       // the g-leg and the column check read f of `parity`
            const double *prow = rows_x ? potx[parity] : poty;    // indexed by the block-local row
            const double *lw = rows_x ? lwx : lwy, *sq = rows_x ? sqx : sqy, *wt = rows_x ? wax : wby;
            const int cs = lane / RG, rg = lane % RG;
            const int lrow0 = warp * RW + rg * R;
            const int row0 = b * RB + lrow0;
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
            for (int r = 0; r < R; ++r) ph[r] = (row0 + r < nrows && form == FORM_DIFF) ? (T)prow[lrow0 + r] : T(0);
            float mx[R];
            double sd[R];
            double m0[R];
#pragma unroll
            for (int r = 0; r < R; ++r) m0[r] = (double)NEG_BIG;
            if constexpr (sizeof(T) == 8 && XF != 0) {
#pragma unroll
                for (int r = 0; r < R; ++r)
                    if (row0 + r < nrows) m0[r] = lw[lrow0 + r] + sq[lrow0 + r] - prow[lrow0 + r];
            }
#pragma unroll 1
            for (int pass = 0; pass < 2; ++pass) {
                if constexpr (sizeof(T) == 4) {
                    if (form == FORM_DOT) stream_f32<DP, CS, FORM_DOT, R, 1>(cols, nullptr, nullptr, nullptr, cp, ncols, xr, ph, tid, cs, mx, sd, stride, trow);
                    else stream_f32<DP, CS, FORM_DIFF, R, 1>(cols, nullptr, nullptr, nullptr, cp, ncols, xr, ph, tid, cs, mx, sd, stride, trow);
                } else {
                    stream_f64<DP, CS, XF, R, 1>(cols, nullptr, nullptr, cp, ncols, xr, tid, cs, m0, mx, sd, stride, trow);
                }
                merge_splits<CS, R>(mx, sd);
                if constexpr (sizeof(T) == 8 && XF != 0) {
                    if (pass == 0) {
                        bool low = false;
#pragma unroll
                        for (int r = 0; r < R; ++r)
                            low = low || (row0 + r < nrows && fabs(m0[r]) < 1.0e7 && !(sd[r] >= 0x1p-20));
                        if (!__syncthreads_or(low ? 1 : 0)) break;
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
            // float64 epilogue, one thread per row; new terms go to every block's copy of the tiles
            unsigned long long term_sum = 0ull;
            for (int lr = tid; lr < RB; lr += UPD_THREADS) {
                const int i = b * RB + lr;
                if (i >= nrows) continue;
                double pnew, term;
                row_math(form, leg != LEG_G, lw[lr], sq[lr], leg != LEG_G ? wt[lr] : 0.0, prow[lr], sc.row_m[lr], sc.row_s[lr],
                         sc.row_h[lr], pnew, term);
                if (leg != LEG_G) {
                    if (!isfinite(term)) block_nf = 1;
                    else term_sum += __double2ull_rn(fmin(term, RSUM_ROW_MAX) * RSUM_SCALE);
                }
                if (leg != LEG_V) {
                    T hi, lo;
                    split_potential<T>(form, pnew, sq[lr], hi, lo);
                    T *dst;
                    if (leg == LEG_F) {
                        potx[parity ^ 1][lr] = pnew;
                        dst = colsX + (size_t)(i / TJ) * STX + (DP + 2 * (parity ^ 1)) * TJ + (i % TJ);
                    } else {
                        poty[lr] = pnew;
                        dst = colsY + (size_t)(i / TJ) * STY + DP * TJ + (i % TJ);
                    }
                    for (int rk = 0; rk < NC; ++rk) { st_cluster<T>(dst, rk, hi); st_cluster<T>(dst + TJ, rk, lo); }
                }
            }
            if (leg != LEG_G) {
                block_nf = __syncthreads_or(block_nf);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) term_sum += __shfl_down_sync(0xffffffffu, term_sum, off);
                unsigned long long *redu = reinterpret_cast<unsigned long long *>(sc.red);
                if (lane == 0) redu[warp] = term_sum;
                __syncthreads();
                if (tid == 0) for (int w = 0; w < UPD_THREADS / 32; ++w) block_sum += redu[w];
            }
        }
        if (leg != LEG_G && tid == 0) {
            const int which = leg == LEG_F ? 0 : 1;
            for (int rk = 0; rk < NC; ++rk) {
                st_cluster<unsigned long long>(&part[which][b], rk, block_sum);
                st_cluster<int>(&part_nf[which][b], rk, block_nf);
            }
        }
        cluster_sync_all();
    };

    int checks = 0, retired_at = 0;
    int leg = LEG_F, it = 0, nf = 0;
    double rr = 0.0, rc = 0.0;
    bool fl = false;
    for (;;) {                                   // one call site for all three kinds of leg
        leg_resident(leg, c.parity);
        if (leg == LEG_G) {
            if (++it >= cycles) break;
            leg = LEG_F;
            continue;
        }
        const int k = c.cycle;
        if (leg == LEG_F) {
            unsigned long long tot = 0ull;
            nf = 0;
            for (int rk = 0; rk < NC; ++rk) { tot += part[0][rk]; nf |= part_nf[0][rk]; }
            rr = (double)tot * (1.0 / RSUM_SCALE);
            const bool audited = lane_audited(P, k, start);
            if (audited && !nf && in_guard_band(P, rr)) {
                // guard band: decide from a float64 re-evaluation of the row residual.  It reads the
                // column potentials from global memory, so the blocks' rows of g go out first.
                for (int lr = tid; lr < RB; lr += UPD_THREADS) {
                    const int i = b * RB + lr;
                    if (i < P.m) P.gam[(size_t)slot * P.mp + i] = poty[lr];
                }
                cluster_sync_all();
                int bad;
                const double *pot_own = potx[c.parity];
                const int r0 = b * RB, r1 = min(r0 + RB, P.n);
                const unsigned long long mine = direct_rows_block<UPD_THREADS / 32>(
                    P, slot, r0, UPD_THREADS / 32, r1, pot_own, r0, reinterpret_cast<unsigned long long *>(sc.red), &bad);
                if (tid == 0) {
                    for (int rk = 0; rk < NC; ++rk) {
                        st_cluster<unsigned long long>(&part[0][b], rk, mine);
                        st_cluster<int>(&part_nf[0][b], rk, bad);
                    }
                }
                cluster_sync_all();
                tot = 0ull;
                for (int rk = 0; rk < NC; ++rk) { tot += part[0][rk]; nf |= part_nf[0][rk]; }
                rr = (double)tot * (1.0 / RSUM_SCALE);
            }
            fl = audited && !nf && rr <= P.tol_screen;
            rc = 0.0;
            if (fl) { leg = LEG_V; continue; }
        } else {
            unsigned long long totc = 0ull;
            for (int rk = 0; rk < NC; ++rk) { totc += part[1][rk]; nf |= part_nf[1][rk]; }
            rc = (double)totc * (1.0 / RSUM_SCALE);
            ++checks;
        }
        const bool vd = !nf && fmax(rr, rc) <= P.tol_stop;
        const bool limit = k - start >= P.max_iter;
        int st = LANE_RUNNING;
        if (nf) st = LANE_NONFINITE;
        else if (fl && vd) st = LANE_DONE;
        else if (limit) st = LANE_ITER_LIMIT;
        if (st != LANE_RUNNING) {
            for (int lr = tid; lr < RB; lr += UPD_THREADS) {
                const int i = b * RB + lr;
                if (i < P.n) P.f_out[(size_t)lane_id * P.n + i] = potx[c.parity][lr] * inv_s;
                if (i < P.m) P.g_out[(size_t)lane_id * P.m + i] = poty[lr] * inv_s;
            }
            if (b == 0 && tid == 0) {
                P.res_row[lane_id] = rr;
                P.res_col[lane_id] = fl ? rc : __longlong_as_double(0x7ff8000000000000LL);
                P.depth[lane_id] = (limit && st != LANE_DONE) ? P.max_iter : k - start;
                P.status[lane_id] = st;
                P.emitted[lane_id] = 1;
            }
            retired_at = k + 1;
            break;
        }
        c.cycle = k + 1;
        c.parity ^= 1;
        leg = LEG_G;
    }
    if (b == 0 && tid == 0) {
        P.ret_at[slot] = retired_at;
        P.n_checks[slot] = checks;
    }
    if (retired_at) return;
    // ---- the lane goes back out: this block's rows of the current potentials and per-point terms
    for (int lr = tid; lr < RB; lr += UPD_THREADS) {
        const int i = b * RB + lr;
        if (i < P.n) {
            const size_t o = (size_t)slot * P.np + i;
            const T *src = colsX + (size_t)(i / TJ) * STX + (DP + 2 * c.parity) * TJ + (i % TJ);
            P.phi[c.parity][o] = potx[c.parity][lr];
            reinterpret_cast<T *>(P.ft[c.parity])[o] = src[0];
            reinterpret_cast<T *>(P.fl[c.parity])[o] = src[TJ];
        }
        if (i < P.m) {
            const size_t o = (size_t)slot * P.mp + i;
            const T *src = colsY + (size_t)(i / TJ) * STY + DP * TJ + (i % TJ);
            P.gam[o] = poty[lr];
            reinterpret_cast<T *>(P.gt)[o] = src[0];
            reinterpret_cast<T *>(P.gl)[o] = src[TJ];
        }
    }
}

}  // namespace skb
