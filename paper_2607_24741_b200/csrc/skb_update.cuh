// Matrix-free Sinkhorn half-step (Eq. 3 in log form) as one streaming kernel.
//
// One launch serves every active lane (grid.y = physical width, grid.x = row blocks):
// the candidate axis of Eq. 2 is a grid axis and nothing is reduced across lanes.
//
// For a row point i of lane t the kernel evaluates, over all column points j,
//     L_i = log2 sum_j 2^(ct_j + r_i . c_j)
// with r, c the scaled coordinates and ct the column term (gt for the f-leg, ft for the
// g-leg), as an online max / sum-of-exp2 reduction: the n x m matrix is never stored.
// Column tiles are staged in shared memory by 16-byte cp.async copies from a
// dimension-major layout; a thread keeps R rows in registers and walks 4 adjacent columns
// per step; with CS > 1 the columns of a tile are split over CS neighbouring lanes of the
// warp and the (max, sum) pairs are merged by xor-shuffles at the end.
//
// Leg-specific epilogues (float64, one per row):
//   LEG_F  phi_new = log2 a + sqx - L;  also the row marginal of the state BEFORE this leg,
//          sum_j pi_ij = a_i 2^(phi_old - phi_new), which is the one-sided row screen of
//          Section "Screen, verify, and compact" obtained for free.
//   LEG_G  gam_new = log2 b + sqy - L  (after it the column marginal equals b, Eq. 4).
//   LEG_V  column marginal of the audited state for screen-positive lanes only,
//          sum_i pi_ij = b_j 2^(gam - gam'), the second half of the two-sided check (Eq. 5).
// The per-CTA L1 partial sums go to scratch; the last CTA of a lane adds them in a fixed
// order and writes the lane's residual and its one flag (screen-positive / verdict).
#pragma once
#include "skb_device.cuh"

namespace skb {

template <int CS> struct TileCols { static constexpr int value = (CS <= 4) ? 128 : (CS == 8 ? 256 : 512); };

template <typename T> struct Vec4 { T v[4]; };

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

template <typename T, int DP, int R, int CS>
__global__ void __launch_bounds__(UPD_THREADS) update_kernel(const Dev P, const int leg)
{
    constexpr int TJ = TileCols<CS>::value;      // columns per shared-memory tile
    constexpr int STEPS = TJ / (4 * CS);         // 4-column groups per thread per tile
    constexpr int RG = 32 / CS;                  // row groups per warp
    constexpr int RW = R * RG;                   // rows per warp
    constexpr int RB = (UPD_THREADS / 32) * RW;  // rows per CTA
    constexpr int EPC = 16 / (int)sizeof(T);     // elements per 16-byte chunk
    constexpr int STAGE = (DP + 1) * TJ;         // elements per stage

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
    const T *rowc = reinterpret_cast<const T *>(rows_x ? P.xs : P.ys) + (size_t)slot * DP * rp;
    const T *colc = reinterpret_cast<const T *>(rows_x ? P.ys : P.xs) + (size_t)slot * DP * cp;
    const T *colt = rows_x ? reinterpret_cast<const T *>(P.gt) + (size_t)slot * cp
                           : reinterpret_cast<const T *>(P.ft[c.parity]) + (size_t)slot * cp;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cs = lane % CS, rg = lane / CS;
    const int row0 = blockIdx.x * RB + warp * RW + rg;   // row r of this thread: row0 + r*RG

    T xr[R][DP];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int i = row0 + r * RG;
#pragma unroll
        for (int k = 0; k < DP; ++k) xr[r][k] = (i < nrows) ? rowc[(size_t)k * rp + i] : T(0);
    }
    T mx[R], ts[R];
    double sd[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { mx[r] = T(NEG_BIG); ts[r] = T(0); sd[r] = 0.0; }

    const int ntiles = (ncols + TJ - 1) / TJ;
    auto load_tile = [&](int t, int stage) {
        T *dst = sm + stage * STAGE;
        const int j0 = t * TJ;
        constexpr int CPR = TJ / EPC;   // chunks per row
        for (int ch = tid; ch < (DP + 1) * CPR; ch += UPD_THREADS) {
            const int k = ch / CPR, j = j0 + (ch % CPR) * EPC;
            T *d = dst + k * TJ + (ch % CPR) * EPC;
            if (j < cp) {
                const T *src = (k < DP) ? colc + (size_t)k * cp + j : colt + j;
                cp_async16(d, src);
            } else {
                const T fill = (k < DP) ? T(0) : T(NEG_BIG);
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
            {
                T ct[4];
                lds4(st + DP * TJ + jj, ct);
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[r][e] = ct[e];
            }
#pragma unroll
            for (int k = 0; k < DP; ++k) {
                T yv[4];
                lds4(st + k * TJ + jj, yv);
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[r][e] = fma(xr[r][k], yv[e], acc[r][e]);
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const T mt = fmax(fmax(acc[r][0], acc[r][1]), fmax(acc[r][2], acc[r][3]));
                if (mt > mx[r] + T(8)) {           // lazy rescale: terms stay below 2^8
                    const T fac = ex2_t(mx[r] - mt);
                    ts[r] *= fac;
                    sd[r] *= (double)fac;
                    mx[r] = mt;
                }
                ts[r] += (ex2_t(acc[r][0] - mx[r]) + ex2_t(acc[r][1] - mx[r])) +
                         (ex2_t(acc[r][2] - mx[r]) + ex2_t(acc[r][3] - mx[r]));
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) { sd[r] += (double)ts[r]; ts[r] = T(0); }
        __syncthreads();
    }

    // merge the CS column splits of each row (xor-shuffle online logsumexp)
    double md[R];
#pragma unroll
    for (int r = 0; r < R; ++r) md[r] = (double)mx[r];
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
            const double pnew = lw[i] + sq[i] - L;
            if (leg == LEG_F) {
                const double pold = P.phi[c.parity][rbase + i];
                term_sum += exp2(lw[i]) * fabs(expm1((pold - pnew) * 0.6931471805599453));
                if (writes) {
                    P.phi[c.parity ^ 1][rbase + i] = pnew;
                    reinterpret_cast<T *>(P.ft[c.parity ^ 1])[rbase + i] = (T)(pnew - sq[i]);
                }
            } else if (leg == LEG_G) {
                if (writes) {
                    P.gam[rbase + i] = pnew;
                    reinterpret_cast<T *>(P.gt)[rbase + i] = (T)(pnew - sq[i]);
                }
            } else {
                const double pold = P.gam[rbase + i];
                term_sum += exp2(lw[i]) * fabs(expm1((pold - pnew) * 0.6931471805599453));
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

template <typename T, int DP, int R, int CS>
inline size_t update_smem_bytes() { return 2 * (size_t)(DP + 1) * TileCols<CS>::value * sizeof(T); }

template <typename T, int DP, int R, int CS>
inline int update_rows_per_cta() { return (UPD_THREADS / 32) * R * (32 / CS); }

}  // namespace skb
