// Large-dimension variant of the streaming update kernel (d > 32, any d up to 1024).
//
// Same contract as update_kernel, but a row's coordinates no longer fit in registers, so both
// operands are staged through shared memory in chunks of KC dimensions: a CTA owns 128 rows,
// walks the columns in tiles of 64, and for every tile accumulates the cross term
// r_i . c_j over all chunks into a 4 x 16 register tile per thread before the online
// max / sum-of-exp2 step.  It is the SIMT fallback and the float64 validation path of the
// dense-contraction workloads; the dot form is the only cost form here.
#pragma once
#include "skb_update.cuh"

namespace skb {

__device__ __forceinline__ void lds4(const float *p, float (&v)[4])
{
    const float4 t = *reinterpret_cast<const float4 *>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void lds4(const double *p, double (&v)[4])
{
    const double2 t0 = *reinterpret_cast<const double2 *>(p);
    const double2 t1 = *reinterpret_cast<const double2 *>(p + 2);
    v[0] = t0.x; v[1] = t0.y; v[2] = t1.x; v[3] = t1.y;
}

constexpr int BIGD_KC = 16;     // dimensions per shared-memory chunk
constexpr int BIGD_RB = 128;    // rows per CTA
constexpr int BIGD_TJ = 64;     // columns per tile

template <typename T, int XF>
__global__ void __launch_bounds__(UPD_THREADS) update_bigd_kernel(const Dev P, const int leg)
{
    constexpr int KC = BIGD_KC, RB = BIGD_RB, TJ = BIGD_TJ, R = 4, CPT = 16;
    constexpr int EPC = 16 / (int)sizeof(T);
    constexpr int STAGE = KC * (RB + TJ);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T *sm = reinterpret_cast<T *>(smem_raw);
    __shared__ double row_s[RB];
    __shared__ float row_m[RB];
    __shared__ float row_h[RB];
    __shared__ double red[UPD_THREADS / 32];

    pdl_enter();
    const Ctl c = *P.ctl;
    if (c.done) return;
    const int slot = blockIdx.y;
    if (slot >= c.n_phys) return;
    if (P.early_exit && P.state[slot] != 0) return;     // early-exit mask arm: a frozen lane costs a launch slot only
    if (leg != LEG_V && c.static_final) return;
    if (leg == LEG_V && !(c.static_final || lane_needs_column_check(P, c, slot))) return;
    const bool rows_x = (leg == LEG_F);
    const int nrows = rows_x ? P.n : P.m, rp = rows_x ? P.np : P.mp;
    const int ncols = rows_x ? P.m : P.n, cp = rows_x ? P.mp : P.np;
    const int i0 = blockIdx.x * RB;
    if (i0 >= nrows) return;
    const int DP = P.DP;
    const T *rowc = reinterpret_cast<const T *>(rows_x ? P.xs : P.ys) + (size_t)slot * DP * rp;
    const T *colc = reinterpret_cast<const T *>(rows_x ? P.ys : P.xs) + (size_t)slot * DP * cp;
    const T *colt = rows_x ? reinterpret_cast<const T *>(P.gt) + (size_t)slot * cp
                           : reinterpret_cast<const T *>(P.ft[c.parity]) + (size_t)slot * cp;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cs = lane / 8, rg = lane % 8;               // 4 column splits x 8 row groups per warp
    const int lrow0 = warp * 32 + rg * R;                 // 4 consecutive CTA-local rows

    const int ntiles = (ncols + TJ - 1) / TJ, nkc = DP / KC, nch = ntiles * nkc;
    auto load_chunk = [&](int ch, int stage) {
        T *A = sm + stage * STAGE, *Bm = A + KC * RB;
        const int t = ch / nkc, k0 = (ch % nkc) * KC, j0 = t * TJ;
        constexpr int CA = RB / EPC, CB = TJ / EPC;
        for (int q = tid; q < KC * (CA + CB); q += UPD_THREADS) {
            const int k = q / (CA + CB), w = q % (CA + CB);
            if (w < CA) {
                const int i = i0 + w * EPC;
                T *d = A + k * RB + w * EPC;
                if (i < rp) cp_async16(d, rowc + (size_t)(k0 + k) * rp + i);
                else { for (int e = 0; e < EPC; ++e) d[e] = T(0); }
            } else {
                const int j = j0 + (w - CA) * EPC;
                T *d = Bm + k * TJ + (w - CA) * EPC;
                if (j < cp) cp_async16(d, colc + (size_t)(k0 + k) * cp + j);
                else { for (int e = 0; e < EPC; ++e) d[e] = T(0); }
            }
        }
    };

    float mx[R];
    double md[R], sd[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { mx[r] = NEG_BIG; md[r] = (double)NEG_BIG; sd[r] = 0.0; }
    T acc[R][CPT];

    load_chunk(0, 0);
    cp_async_commit();
    for (int ch = 0; ch < nch; ++ch) {
        if (ch + 1 < nch) {
            load_chunk(ch + 1, (ch + 1) & 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const T *A = sm + (ch & 1) * STAGE, *Bm = A + KC * RB;
        if (ch % nkc == 0) {
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int e = 0; e < CPT; ++e) acc[r][e] = T(0);
        }
#pragma unroll 4
        for (int k = 0; k < KC; ++k) {
            T xa[4];
            lds4(A + k * RB + lrow0, xa);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                T yb[4];
                lds4(Bm + k * TJ + (q * 4 + cs) * 4, yb);
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[r][q * 4 + e] = fma(xa[r], yb[e], acc[r][q * 4 + e]);
            }
        }
        if (ch % nkc == nkc - 1) {
            // the tile's arguments are complete: add the column terms, then the online update
            const int j0 = (ch / nkc) * TJ;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int j = j0 + (q * 4 + cs) * 4 + e;
                    const T ct = (j < cp) ? colt[j] : T(NEG_BIG);
#pragma unroll
                    for (int r = 0; r < R; ++r) acc[r][q * 4 + e] += ct;
                }
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                T mt = acc[r][0];
#pragma unroll
                for (int e = 1; e < CPT; ++e) mt = fmax(mt, acc[r][e]);
                if ((double)mt > md[r] + 8.0) {
                    const float mn = ceilf((float)mt) + 1.0f;
                    sd[r] *= (double)pow2i(mx[r] - mn);
                    mx[r] = mn;
                    md[r] = (double)mn;
                }
                if (sizeof(T) == 4 || XF) {
                    float ts = 0.f;
#pragma unroll
                    for (int e = 0; e < CPT; ++e) ts += ex2_fast((float)(acc[r][e] - (T)md[r]));
                    sd[r] += (double)ts;
                } else {
#pragma unroll
                    for (int e = 0; e < CPT; ++e) sd[r] += exp2((double)acc[r][e] - md[r]);
                }
            }
        }
        __syncthreads();
    }

    // merge the 4 column splits (lanes 8 apart); maxima are integers, scalings exact
#pragma unroll
    for (int off = 8; off < 32; off <<= 1) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float mo = __shfl_xor_sync(0xffffffffu, mx[r], off);
            const double so = __shfl_xor_sync(0xffffffffu, sd[r], off);
            const float mn = fmaxf(mx[r], mo);
            sd[r] = sd[r] * (double)pow2i(mx[r] - mn) + so * (double)pow2i(mo - mn);
            mx[r] = mn;
        }
    }
    if (cs == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) { row_m[lrow0 + r] = mx[r]; row_s[lrow0 + r] = sd[r]; row_h[lrow0 + r] = 0.f; }
    }
    __syncthreads();
    finish_rows<T, RB>(P, c, leg, slot, (int)FORM_DOT, row_m, row_s, row_h, red, (int)blockIdx.x * RB);
}

}  // namespace skb
