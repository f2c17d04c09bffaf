// Tensor-core variants of the update kernel for bf16 point clouds with a deep cross term
// (d a multiple of 64, 64 <= d <= 512): the only place on the path that is a dense
// contraction.
//
// For a block of 128 row points a CTA computes S = R . C^T against tiles of column points
// with tcgen05.mma (bf16 operands, fp32 accumulators in tensor memory), then
// log2 pi_ij = 2 s S_ij + ct_j and the same online max / sum-of-exp2 reduction and float64
// epilogue as the SIMT kernels (dot form).  Operands come from pre-tiled copies (every
// 128-point x 64-dimension chunk is one contiguous 16 KB block in the workspace, which TMA
// streams at about twice the rate of 1 KB-strided rows; 128-byte swizzle; points past the end
// are stored as zeros).
//
// Two kernels:
//   update_tc_kernel        d <= 256: one CTA per row block, 128-column tiles, a two-stage ring,
//                           small enough for two CTAs per SM
//   update_tc_pair_kernel   d > 256: persistent clusters of two CTAs (tcgen05 cta_group::2, M = 256,
//                           N = 256), described at its definition
// Warp roles of both: warps 0-7 epilogue (thread <-> row <-> TMEM lane; warps 0-3 take the even
// 32-column chunks of a tile, warps 4-7 the odd ones; tcgen05.ld one chunk ahead, packed fp32
// arithmetic, no shuffles), one producer warp (one lane issues the TMA loads: the row block
// once, riding on the first tile's barriers, then column chunks through the ring), one MMA
// warp (allocates tensor memory for two accumulators; one lane issues 4 x K=16 MMAs per
// 64-dimension chunk and commits to the ring's empty barriers and to the accumulator-full
// barrier, so the next tile's MMAs overlap this tile's exponentials).
// Every mbarrier wait is bounded by a clock budget; on expiry the kernel raises ERR_WAIT in
// the control block, all roles leave their loops, tensor memory is freed and the kernel
// returns (the host reports SKB_ERR_CUDA).
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdio>

#include "skb_update.cuh"
#include "skb_host.h"

namespace skb {

constexpr int TC_EPI_WARPS = 8;                            // two per scheduler: lanes (w & 3), column half (w >> 2)
constexpr int TC_EPI_THREADS = TC_EPI_WARPS * 32;
constexpr int TC_THREADS = TC_EPI_THREADS + 64;            // + producer warp + MMA warp
constexpr int TC_MAX_STAGES = 4;
constexpr int TC_BM = 128, TC_BK = 64;
constexpr uint32_t TC_CHUNK = TC_BM * TC_BK * 2;          // 16 KB: 128 points x 64 bf16
constexpr long long TC_WAIT_CLOCKS = 2000000000LL;        // ~1 s: budget of every bounded wait of the update kernels

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t a, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t a)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t a, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(a), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t a, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(a), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the budget ran out or another role already gave up.
// The budget is an argument (the update kernels use the constant, the self-test its own short one):
// a writable global would let a self-test on one stream shorten the waits of a solve on another.
__device__ __forceinline__ bool mbar_wait(uint32_t a, uint32_t parity, volatile int *abort_flag,
                                          const long long budget = TC_WAIT_CLOCKS)
{
    if (mbar_try_wait(a, parity)) return true;          // the common case costs no clock read
    const long long t0 = clock64();
    while (!mbar_try_wait(a, parity)) {
        if (*abort_flag) return false;
        if (clock64() - t0 > budget) { *abort_flag = 1; return false; }
    }
    return true;
}
// one pre-tiled chunk (128 points x 64 bf16, contiguous 16 KB in global memory) -> shared memory
#ifdef SKB_TC_DEBUG
#define TC_TIMED_WAIT(acc, call) ({ const long long _t = clock64(); const bool _r = (call); (acc) += clock64() - _t; _r; })
#else
#define TC_TIMED_WAIT(acc, call) (call)
#endif
__device__ __forceinline__ void tma_load_chunk(uint32_t dst, const CUtensorMap *tm, int row, uint32_t mbar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(0), "r"(row), "r"(mbar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t mbar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane; asynchronous until tc_ld_wait()
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// Completes every load this thread has issued.  The registers pass through the statement so
// that the compiler cannot move a use of them above it.
__device__ __forceinline__ void tc_ld_wait(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}

// Online max / sum-of-exp2 over one 32-column chunk of a row: arg = 2 s S + ct_j, computed
// on column pairs with packed fp32 instructions.  The running reference mx is NOT updated on
// the fast path: the exponentials are taken against the reference as it stands and only their
// sum is tested.  A sum above 2^10 (some argument more than ~5 above the reference, which
// would cost exponent accuracy; a reference of minus infinity gives an infinite sum) sends
// the chunk through the exact path: maximum, integer-valued new reference, exact rescale.
// The reference therefore is always the ceiling of a true argument of this row, so terms can
// never all underflow.
__device__ __forceinline__ void tc_reduce_chunk(const uint32_t (&r)[32], const float *gt, const float two_s,
                                                float &mx, float &ts, double &sd)
{
    u64 v[16];
    const u64 s2 = pack2(two_s, two_s);
    const u64 nm = pack2(-mx, -mx);
    u64 acc[2] = {0ull, 0ull};
#pragma unroll
    for (int q = 0; q < 32; q += 4) {
        const float4 g = *reinterpret_cast<const float4 *>(gt + q);
        v[q / 2] = fma2(pack2(__uint_as_float(r[q]), __uint_as_float(r[q + 1])), s2, pack2(g.x, g.y));
        v[q / 2 + 1] = fma2(pack2(__uint_as_float(r[q + 2]), __uint_as_float(r[q + 3])), s2, pack2(g.z, g.w));
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float d0, d1;
            unpack2(add2(v[q / 2 + h], nm), d0, d1);
            acc[h] = add2(acc[h], pack2(ex2_fast(d0), ex2_fast(d1)));
        }
    }
    float a0, a1, a2, a3;
    unpack2(acc[0], a0, a1);
    unpack2(acc[1], a2, a3);
    float sc = (a0 + a1) + (a2 + a3);
    if (!(sc <= 1024.f)) {
        float m4[4] = {NEG_BIG, NEG_BIG, NEG_BIG, NEG_BIG};
#pragma unroll
        for (int q = 0; q < 16; q += 2) {
            float x0, x1, x2, x3;
            unpack2(v[q], x0, x1);
            unpack2(v[q + 1], x2, x3);
            m4[0] = fmaxf(m4[0], x0); m4[1] = fmaxf(m4[1], x1);
            m4[2] = fmaxf(m4[2], x2); m4[3] = fmaxf(m4[3], x3);
        }
        const float mt = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        if (mt > mx) {                                  // always, unless the sum itself was not finite
            const float mn = ceilf(mt);
            const float fac = pow2i(mx - mn);
            ts *= fac;
            sd *= (double)fac;
            mx = mn;
        }
        float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int q = 0; q < 16; q += 2) {
            float x0, x1, x2, x3;
            unpack2(v[q], x0, x1);
            unpack2(v[q + 1], x2, x3);
            s4[0] += ex2_fast(x0 - mx); s4[1] += ex2_fast(x1 - mx);
            s4[2] += ex2_fast(x2 - mx); s4[3] += ex2_fast(x3 - mx);
        }
        sc = (s4[0] + s4[1]) + (s4[2] + s4[3]);
    }
    ts += sc;
}

// One accumulator tile of BN columns: this warp's half of the 32-column chunks (even or odd),
// the next chunk's tensor-memory load in flight while the current one is reduced.
template <int BN>
__device__ __forceinline__ void tc_reduce_tile(const uint32_t taddr, const float *gt, const int half, const float two_s,
                                               float &mx, float &ts, double &sd)
{
    constexpr int NCH = BN / 64;                   // chunks per warp
    static_assert(NCH % 2 == 0, "chunks are processed in pairs");
    uint32_t ra[32], rb[32];
    tc_ld32_issue(taddr + (uint32_t)(half * 32), ra);
    tc_ld_wait(ra);
#pragma unroll
    for (int i = 0; i < NCH; i += 2) {
        const int c0 = (2 * i + half) * 32, c1 = c0 + 64;
        tc_ld32_issue(taddr + (uint32_t)c1, rb);
        tc_reduce_chunk(ra, gt + c0, two_s, mx, ts, sd);
        tc_ld_wait(rb);
        if (i + 2 < NCH) tc_ld32_issue(taddr + (uint32_t)(c1 + 64), ra);
        tc_reduce_chunk(rb, gt + c1, two_s, mx, ts, sd);
        if (i + 2 < NCH) tc_ld_wait(ra);
    }
}

// Merges the two column halves of every row (warps 4-7 hand theirs to warps 0-3 through `xm`,
// `xs`: 128 floats and 128 doubles of shared memory nobody else uses any more) and leaves the
// row results where finish_rows expects them.  Called by all epilogue threads.
__device__ __forceinline__ void tc_merge_halves(const int e, const float mx, const double sd, const bool ok,
                                                float *xm, double *xs, float *row_m, double *row_s, float *row_h)
{
    const int row = e & 127;
    if (e >= 128) { xm[row] = mx; xs[row] = ok ? sd : __longlong_as_double(0x7ff8000000000000LL); }
    asm volatile("bar.sync 1, 256;" ::: "memory");     // also: every row is done with the column terms
    if (e < 128) {
        const float mo = xm[row];
        const double so = xs[row];
        const float mn = fmaxf(mx, mo);
        row_m[row] = mn;
        row_s[row] = ok ? sd * (double)pow2i(mx - mn) + so * (double)pow2i(mo - mn) : __longlong_as_double(0x7ff8000000000000LL);
        row_h[row] = 0.f;
    }
}
// shared-memory matrix descriptor: K-major tile, rows of 64 bf16 (128 B), 128-byte swizzle,
// 8-row groups 1024 B apart
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = 128
__host__ __device__ constexpr uint32_t tc_idesc(int bn) { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24); }

template <int TC_STAGES, int TC_BN>
__global__ void __launch_bounds__(TC_THREADS, TC_BN == 128 ? 2 : 1)
update_tc_kernel(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmy, const Dev P, const int leg)
{
    extern __shared__ __align__(1024) unsigned char smem_tc[];
    __shared__ __align__(8) unsigned long long bars[2 * TC_MAX_STAGES + 5];
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;
    // column terms of two tiles while streaming; the per-row results afterwards (same bytes)
    __shared__ __align__(16) unsigned char small_buf[2 * TC_BN * 4 > 2048 ? 2 * TC_BN * 4 : 2048];
    float (*gts)[TC_BN] = reinterpret_cast<float (*)[TC_BN]>(small_buf);
    double *row_s = reinterpret_cast<double *>(small_buf);
    float *row_m = reinterpret_cast<float *>(small_buf + 1024);
    float *row_h = reinterpret_cast<float *>(small_buf + 1536);
    constexpr uint32_t STAGE_BYTES = (TC_BN / 128) * TC_CHUNK;     // one or two 128-point chunks per stage
    __shared__ double red[TC_THREADS / 32];

    pdl_enter();
    const Ctl c = *P.ctl;
    if (c.done) return;
    const int slot = blockIdx.y;
    if (slot >= c.n_phys) return;
    if (P.early_exit && P.state[slot] != 0) return;     // early-exit mask arm: a frozen lane costs a launch slot only
    if (leg != LEG_V && c.static_final) return;
    if (leg == LEG_V && !(c.static_final || lane_needs_column_check(P, c, slot))) return;
    const bool rows_x = (leg == LEG_F);
    const int nrows = rows_x ? P.n : P.m;
    const int ncols = rows_x ? P.m : P.n, cp = rows_x ? P.mp : P.np;
    const int i0 = blockIdx.x * TC_BM;
    if (i0 >= nrows) return;
    const CUtensorMap *tm_row = rows_x ? &tmx : &tmy, *tm_col = rows_x ? &tmy : &tmx;
    const float *colt = rows_x ? reinterpret_cast<const float *>(P.gt) + (size_t)slot * cp
                               : reinterpret_cast<const float *>(P.ft[c.parity]) + (size_t)slot * cp;
    const int nkc = P.d / TC_BK;
    const int ntiles = (ncols + TC_BN - 1) / TC_BN;
    // chunk index of this CTA's row block and of the lane's first column tile in the tiled copies
    const int nrt = (nrows + TC_BM - 1) / TC_BM;
    const int row_tile0 = (slot * nrt + (int)blockIdx.x) * nkc;
    const int nct128 = (ncols + 127) / 128;                     // 128-point tiles of the column operand
    const int col_tile0 = slot * nct128 * nkc;
    const float two_s = (float)(2.0 * P.scale[slot]);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // shared memory: row block (nkc chunks) then the column ring; 1024-byte aligned for the swizzle
    const uint32_t sbase = (smem_u32(smem_tc) + 1023u) & ~1023u;
    const uint32_t sA = sbase, sB = sbase + (uint32_t)nkc * TC_CHUNK;
    const uint32_t b_full = smem_u32(&bars[0]), b_empty = smem_u32(&bars[TC_STAGES]);
    const uint32_t b_a = smem_u32(&bars[2 * TC_STAGES]);
    const uint32_t b_tfull = smem_u32(&bars[2 * TC_STAGES + 1]), b_tempty = smem_u32(&bars[2 * TC_STAGES + 3]);

    if (tid == 0) {
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(b_full + 8 * s, 1); mbar_init(b_empty + 8 * s, 1); }
        mbar_init(b_a, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(b_tfull + 8 * b, 1); mbar_init(b_tempty + 8 * b, TC_EPI_THREADS); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == TC_EPI_WARPS + 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&tmem_holder)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_holder;
    volatile int *ab = &abort_flag;

    float mx = NEG_BIG;
    double sd = 0.0;
    long long dbg_w0 = 0, dbg_w1 = 0;   // clocks spent in waits (debug builds)
    const long long dbg_t0 = clock64();
    (void)dbg_w0; (void)dbg_w1; (void)dbg_t0;

    if (warp == TC_EPI_WARPS) {
        // ---------------- producer
        if (lane == 0) {
            // the row block rides on the first tile's ring barriers, chunk by chunk, so the first
            // MMAs start as soon as one chunk of each operand has landed
            int it = 0;
            for (int t = 0; t < ntiles && !*ab; ++t) {
                for (int kc = 0; kc < nkc; ++kc, ++it) {
                    const int s = it % TC_STAGES;
                    if (it >= TC_STAGES && !TC_TIMED_WAIT(dbg_w0, mbar_wait(b_empty + 8 * s, ((it / TC_STAGES) - 1) & 1, ab))) break;
                    mbar_expect_tx(b_full + 8 * s, t == 0 ? STAGE_BYTES + TC_CHUNK : STAGE_BYTES);
                    if (t == 0) tma_load_chunk(sA + kc * TC_CHUNK, tm_row, (row_tile0 + kc) * TC_BM, b_full + 8 * s);
#pragma unroll
                    for (int h = 0; h < TC_BN / 128; ++h) {
                        // 128-point tile index of this half of the column tile; tiles past the end read as zeros
                        const int pt = t * (TC_BN / 128) + h;
                        if (pt < nct128)
                            tma_load_chunk(sB + s * STAGE_BYTES + h * TC_CHUNK, tm_col, (col_tile0 + pt * nkc + kc) * 128, b_full + 8 * s);
                        else
                            tma_load_chunk(sB + s * STAGE_BYTES + h * TC_CHUNK, tm_col, 0x7fffff80, b_full + 8 * s);
                    }
                }
            }
        }
    } else if (warp == TC_EPI_WARPS + 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            bool ok = true;
            int it = 0;
            for (int t = 0; t < ntiles && ok; ++t) {
                const int buf = t & 1;
                if (t >= 2) ok = TC_TIMED_WAIT(dbg_w1, mbar_wait(b_tempty + 8 * buf, ((t >> 1) - 1) & 1, ab));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem + (uint32_t)buf * TC_BN;
                for (int kc = 0; kc < nkc && ok; ++kc, ++it) {
                    const int s = it % TC_STAGES;
                    ok = TC_TIMED_WAIT(dbg_w0, mbar_wait(b_full + 8 * s, (it / TC_STAGES) & 1, ab));
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k) {
                        const uint64_t bd = tc_desc(sB + s * STAGE_BYTES + k * 32);
                        const uint64_t ad = tc_desc(sA + kc * TC_CHUNK + k * 32);
                        tc_mma(d_tmem, ad, bd, tc_idesc(TC_BN), (kc | k) ? 1u : 0u);
                    }
                    tc_commit(b_empty + 8 * s);             // frees the ring stage when these MMAs retire
                }
                if (ok) tc_commit(b_tfull + 8 * buf);       // accumulator complete
            }
        }
    } else {
        // ---------------- epilogue: thread e <-> row (e & 127) <-> TMEM lane (e & 127); warps 0-3 take
        // the even 32-column chunks of every tile, warps 4-7 the odd ones
        const int e = tid, half = warp >> 2;
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = true;
        float ts = 0.f;
        static_assert(TC_BN <= TC_EPI_THREADS, "one column term per epilogue thread and tile");
        float g_next = (e < TC_BN && e < cp) ? colt[e] : NEG_BIG;       // column term, one tile ahead
        for (int t = 0; t < ntiles && ok; ++t) {
            const int buf = t & 1;
            if (e < TC_BN) {
                gts[buf][e] = g_next;
                const int j = (t + 1) * TC_BN + e;
                g_next = (t + 1 < ntiles && j < cp) ? colt[j] : NEG_BIG;
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            ok = TC_TIMED_WAIT(dbg_w0, mbar_wait(b_tfull + 8 * buf, (t >> 1) & 1, ab));
            if (!ok) break;
            tc_fence_after();
            tc_reduce_tile<TC_BN>(lane_base + (uint32_t)(buf * TC_BN), gts[buf], half, two_s, mx, ts, sd);
            sd += (double)ts;
            ts = 0.f;
            tc_fence_before();
            mbar_arrive(b_tempty + 8 * buf);                // all rows have read this accumulator
        }
        // the ring is idle by now: its first bytes carry the second half's partial results
        tc_merge_halves(e, mx, sd, ok, reinterpret_cast<float *>(smem_tc + (sB - smem_u32(smem_tc)) + 1024),
                        reinterpret_cast<double *>(smem_tc + (sB - smem_u32(smem_tc))), row_m, row_s, row_h);
    }
    if (abort_flag) {
        // a wait ran out: give copies that may still be in flight time to land in this CTA's
        // shared memory before it is released (bounded: ~0.1 ms)
        const long long t0 = clock64();
        while (clock64() - t0 < 200000LL) { }
    }
#ifdef SKB_TC_DEBUG
    if (blockIdx.x == 1 && blockIdx.y == 3 && leg == LEG_F && (lane == 0) && (warp == 0 || warp == 4 || warp >= TC_EPI_WARPS))
        printf("[tc dbg] warp %d: total %lld clk, wait0 %lld, wait1 %lld (producer: empty; mma: full, tmem-empty; epilogue: tmem-full) tiles %d chunks/tile %d\n",
               warp, clock64() - dbg_t0, dbg_w0, dbg_w1, ntiles, nkc);
#endif
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == TC_EPI_WARPS + 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
    }
    if (abort_flag) {
        if (tid == 0) atomicOr(&P.ctl->error, ERR_WAIT);
    }
    finish_rows<float, TC_BM, TC_THREADS>(P, c, leg, slot, (int)FORM_DOT, row_m, row_s, row_h, red, (int)blockIdx.x * TC_BM);
}

// ---------------------------------------------------------------- CTA-pair variant
// Two CTAs of a cluster (two SMs) work on 256 consecutive row points of one lane with
// tcgen05.mma.cta_group::2 (M = 256: 128 rows per CTA, N = 256).  Each CTA keeps its own 128-row
// block resident and streams only ITS half of every 256-column tile (128 points x 64 dimensions
// = 16 KB per ring stage); the tensor cores of both SMs read both halves.  Per SM that halves
// the L2 -> shared-memory traffic of the column operand and leaves room for a deeper ring
// (six stages beside a 128 KB row block), which is what the single-CTA kernel is short of.
//
// Barriers (same offsets in both CTAs):  full[s]  lives in the leader (cluster rank 0): one
// arrival by the leader's producer, which expects the bytes of BOTH CTAs' copies; the peer's
// copies complete on the leader's barrier.  empty[s] and tfull[b] are per CTA: the leader's MMA
// thread commits to its own and to the peer's.  tempty[b] lives in the leader and counts the
// 256 epilogue threads of the pair (the peer's arrive remotely).  Every wait is bounded as in
// the single-CTA kernel; the two cluster-wide barriers are plain hardware barriers that every
// thread of both CTAs reaches on every path (the early exits above them depend on the lane
// only, which the pair shares).
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// as tma_load_chunk, but the completion barrier may live in the peer CTA of the pair
__device__ __forceinline__ void tma_load_chunk_pair(uint32_t dst, const CUtensorMap *tm, int row, uint32_t mbar_cluster)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(0), "r"(row), "r"(mbar_cluster) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t mbar_cluster)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar_cluster) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// instruction descriptor of the pair: D fp32, A and B bf16 K-major, M = 256 (two CTAs), N = 256
__host__ __device__ constexpr uint32_t tc_idesc_pair() { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24); }

constexpr int TC2_BN = 256;               // columns per accumulator tile
constexpr int TC2_MAX_STAGES = 8;
constexpr int TC2_FILE_WARPS = 4;               // one thread per row of an item for the float64 epilogue
constexpr int TC2_THREADS = TC_THREADS + 32 * TC2_FILE_WARPS;

// all-threads AND over the 256 epilogue threads (they must leave their loops together)
__device__ __forceinline__ bool epi_all(const bool ok)
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\tbar.red.and.pred q, 3, 256, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(r) : "r"((uint32_t)ok) : "memory");
    return r != 0;
}

// the same over the 128 threads of the filing warps
__device__ __forceinline__ bool file_all(const bool ok)
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\tbar.red.and.pred q, 5, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(r) : "r"((uint32_t)ok) : "memory");
    return r != 0;
}

// The kernel is PERSISTENT and TILE-BALANCED.  The work of a launch is the sequence of units
// (lane, pair of row blocks, group of column tiles), `upi` units per row-block pair; the grid
// holds one cluster per SM pair and cluster c takes the units [c U / C, (c+1) U / C).  A run
// of units of one row-block pair is a SEGMENT: the cluster loads the pair's row blocks once and
// reduces the segment's column tiles.  Barrier set-up, tensor-memory allocation, the first
// loads of a segment, the exponentials of its last tile and its float64 epilogue all overlap
// the MMAs of the neighbouring segments; the ring, the accumulator buffers and their barrier
// phases simply run on.  A row-block chunk of the NEXT segment may overwrite the resident copy
// as soon as the ring stage it travels with has been released, because MMAs retire in order
// and the ring (nstages <= d/64 stages) is not longer than a tile: the release of that stage
// implies that the last tile's MMAs on the same chunk have retired.
//
// Every unit's row results (maximum, sum; one pair per column half) go to global scratch, and
// a row block is finished by merging ALL its units' results in unit order: the value does not
// depend on how the units were shared out, so every mode and every width gives the same bits.
// A row block whose units went to several clusters is finished by whichever of them arrives
// last (each adds its unit count to the block's arrival word after a fence).
// column tiles per unit: at most TC_MAX_SPLIT units per row-block pair, and two tiles per unit
// where there are that many (every unit starts its reduction cold, which costs one exact-path
// chunk per warp)
__host__ __device__ constexpr int tc_unit_tiles(int ntiles)
{
    const int g = (ntiles + TC_MAX_SPLIT - 1) / TC_MAX_SPLIT;
    return g < 2 && ntiles >= 2 ? 2 : g;
}
struct Seg { int slot, pb, t0, t1, fu, nu; };
struct SegIter {
    int u, u_end, upi, g, npair, ntiles;
    __device__ __forceinline__ bool next(Seg &s)
    {
        if (u >= u_end) return false;
        const int item = u / upi;
        s.fu = u - item * upi;
        s.nu = min(upi - s.fu, u_end - u);
        u += s.nu;
        s.slot = item / npair;
        s.pb = item - s.slot * npair;
        s.t0 = s.fu * g;
        s.t1 = min(ntiles, (s.fu + s.nu) * g);
        return true;
    }
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC2_THREADS, 1)
update_tc_pair_kernel(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmy, const Dev P, const int leg,
                      const int nstages)
{
    extern __shared__ __align__(1024) unsigned char smem_tc[];
    __shared__ __align__(8) unsigned long long bars[2 * TC2_MAX_STAGES + 6];
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;
    __shared__ unsigned arrival;                           // filing warps: the arrival word before this part's add
    __shared__ __align__(16) float gts[TC2_BN];            // column terms of the tile being reduced
    __shared__ unsigned long long red[TC2_FILE_WARPS];

    // Set-up that touches nothing an earlier kernel writes comes BEFORE the wait for that kernel:
    // with programmatic dependent launch it overlaps the predecessor's tail (on SMs that are free).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_rank();
    const bool leader = (rank == 0);
    const uint32_t b_full = smem_u32(&bars[0]), b_empty = smem_u32(&bars[TC2_MAX_STAGES]);
    const uint32_t b_tfull = smem_u32(&bars[2 * TC2_MAX_STAGES]), b_tempty = b_tfull + 16;
    const uint32_t b_box_full = b_tfull + 32, b_box_empty = b_tfull + 40;
    // the same barriers seen in the leader's / the peer's shared memory
    const uint32_t b_full_leader = map_to_cta(b_full, 0);
    const uint32_t b_tempty_leader = map_to_cta(b_tempty, 0);
    const uint32_t b_empty_peer = map_to_cta(b_empty, 1);
    const uint32_t b_tfull_peer = map_to_cta(b_tfull, 1);
    if (tid == 0) {
        for (int s = 0; s < nstages; ++s) mbar_init(b_full + 8 * s, 1);
        for (int q = 0; q < nstages; ++q) mbar_init(b_empty + 8 * q, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(b_tfull + 8 * b, 1); mbar_init(b_tempty + 8 * b, 2 * TC_EPI_WARPS); }
        mbar_init(b_box_full, 1); mbar_init(b_box_empty, TC2_FILE_WARPS);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == TC_EPI_WARPS + 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&tmem_holder)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_barrier();                                  // both CTAs' barriers exist before anything remote touches them
    tc_fence_after();
    asm volatile("griddepcontrol.wait;" ::: "memory");  // from here on: data of the kernels before this one

    const Ctl c = *P.ctl;
    // nothing to do (batch finished, or STATIC's closing pass, which runs the column check only):
    // an empty unit range, and the common exit below
    const bool idle = c.done || (leg != LEG_V && c.static_final);
    const bool rows_x = (leg == LEG_F);
    const int nrows = rows_x ? P.n : P.m;
    const int ncols = rows_x ? P.m : P.n, cp = rows_x ? P.mp : P.np;
    const int nrt = (nrows + TC_BM - 1) / TC_BM;
    const int npair = (nrt + 1) / 2;                       // row-block pairs per lane (the last may be half empty)
    const CUtensorMap *tm_row = rows_x ? &tmx : &tmy, *tm_col = rows_x ? &tmy : &tmx;
    const int nkc = P.d / TC_BK;
    const int ntiles = (ncols + TC2_BN - 1) / TC2_BN;
    const int nct128 = (ncols + 127) / 128;
    // units: groups of g column tiles, at most TC_MAX_SPLIT per row-block pair
    const int g = tc_unit_tiles(ntiles);
    const int upi = (ntiles + g - 1) / g;
    const int U = idle ? 0 : c.n_phys * npair * upi;
    const int ncl_grid = (int)gridDim.x >> 1, ncl = ncl_grid < U ? ncl_grid : U, cl = (int)blockIdx.x >> 1;
    SegIter it0;
    it0.upi = upi; it0.g = g; it0.npair = npair; it0.ntiles = ntiles;
    it0.u = cl < ncl ? (int)((long long)cl * U / ncl) : 0;
    it0.u_end = cl < ncl ? (int)((long long)(cl + 1) * U / ncl) : 0;

    const uint32_t sbase = (smem_u32(smem_tc) + 1023u) & ~1023u;
    const uint32_t sA = sbase, sB = sbase + (uint32_t)nkc * TC_CHUNK;
    const uint32_t tmem = tmem_holder;
    volatile int *ab = &abort_flag;
#ifdef SKB_TC_DEBUG
    long long dbg_w0 = 0, dbg_w1 = 0;   // clocks spent in waits
    const long long dbg_t0 = clock64();
#endif

    // every role walks the same segments and skips the same ones (the column check only
    // visits lanes that the screen flagged)
    SegIter it = it0;
    Seg sg;
#define TC2_SKIP(slot) ((leg == LEG_V && !(c.static_final || lane_needs_column_check(P, c, slot))) || (P.early_exit && P.state[slot] != 0))

    if (warp == TC_EPI_WARPS) {
        // ---------------- producer (one per CTA): own row block once per segment, own half of every column tile
        if (lane == 0) {
            int s = 0; uint32_t ph = 0;
            bool first_round = true, go = true;
            while (go && it.next(sg)) {
                if (TC2_SKIP(sg.slot)) continue;
                const int rb = 2 * sg.pb + (int)rank;
                const bool ghost = rb >= nrt;                  // odd number of row blocks: no rows for the pair's second CTA
                const int row_tile0 = (sg.slot * nrt + rb) * nkc;
                const int col_tile0 = sg.slot * nct128 * nkc;
                for (int t = sg.t0; t < sg.t1 && go; ++t) {
                    for (int kc = 0; kc < nkc; ++kc) {
                        if (!first_round && !TC_TIMED_WAIT(dbg_w0, mbar_wait(b_empty + 8 * s, ph ^ 1u, ab))) { go = false; break; }
                        if (leader) mbar_expect_tx(b_full + 8 * s, t == sg.t0 ? 4 * TC_CHUNK : 2 * TC_CHUNK);
                        if (t == sg.t0)
                            tma_load_chunk_pair(sA + kc * TC_CHUNK, tm_row, ghost ? 0x7fffff80 : (row_tile0 + kc) * TC_BM, b_full_leader + 8 * s);
                        const int pt = t * 2 + (int)rank;              // this CTA's 128-point tile of the column operand
                        tma_load_chunk_pair(sB + s * TC_CHUNK, tm_col, pt < nct128 ? (col_tile0 + pt * nkc + kc) * 128 : 0x7fffff80,
                                            b_full_leader + 8 * s);
                        if (++s == nstages) { s = 0; ph ^= 1u; first_round = false; }
                    }
                }
                if (*ab) go = false;
            }
        }
    } else if (warp == TC_EPI_WARPS + 1) {
        // ---------------- MMA issuer (leader only)
        if (lane == 0 && leader) {
            bool ok = true;
            int s = 0; uint32_t ph = 0;
            int tg = 0;                                         // tiles issued so far: accumulator buffer and phase
            const uint64_t adesc0 = tc_desc(sA), bdesc0 = tc_desc(sB);   // the address field counts 16-byte units
            while (ok && it.next(sg)) {
                if (TC2_SKIP(sg.slot)) continue;
                for (int t = sg.t0; t < sg.t1 && ok; ++t, ++tg) {
                    const int buf = tg & 1;
                    if (tg >= 2) ok = TC_TIMED_WAIT(dbg_w1, mbar_wait(b_tempty + 8 * buf, ((tg >> 1) - 1) & 1, ab));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem + (uint32_t)buf * TC2_BN;
                    uint64_t ad = adesc0;
                    for (int kc = 0; kc < nkc && ok; ++kc, ad += TC_CHUNK >> 4) {
                        ok = TC_TIMED_WAIT(dbg_w0, mbar_wait(b_full + 8 * s, ph, ab));
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t bd = bdesc0 + (uint64_t)(s * (TC_CHUNK >> 4));
                        // four K = 16 slices of the 64-dimension chunk: 32 bytes apart inside the swizzle atom
                        tc_mma_pair(d_tmem, ad, bd, tc_idesc_pair(), kc ? 1u : 0u);
                        tc_mma_pair(d_tmem, ad + 2, bd + 2, tc_idesc_pair(), 1u);
                        tc_mma_pair(d_tmem, ad + 4, bd + 4, tc_idesc_pair(), 1u);
                        tc_mma_pair(d_tmem, ad + 6, bd + 6, tc_idesc_pair(), 1u);
                        tc_commit_pair(b_empty + 8 * s);        // both producers may refill this stage
                        tc_commit_pair(b_empty_peer + 8 * s);
                        if (++s == nstages) { s = 0; ph ^= 1u; }
                    }
                    if (ok) { tc_commit_pair(b_tfull + 8 * buf); tc_commit_pair(b_tfull_peer + 8 * buf); }
                }
            }
        }
    } else if (warp >= TC_EPI_WARPS + 2) {
        // ---------------- filing warps (one thread per row): take each segment's merged row results
        // (maximum, sum) from the epilogue warps and do everything that is slow and serial off
        // their critical path: the hand-over between the parts of a shared row block, the merge of
        // all units in unit order, the float64 epilogue of the rows and their residual terms
        const int fw = warp - (TC_EPI_WARPS + 2), row = fw * 32 + lane;
        int k = 0;
        while (it.next(sg)) {
            if (TC2_SKIP(sg.slot)) continue;
            const int slot = sg.slot, rb = 2 * sg.pb + (int)rank;
            if (rb >= nrt) continue;                                    // no rows, no message
            int got = 0;
            if (lane == 0) got = mbar_wait(b_box_full, k & 1, ab) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!file_all(got != 0)) break;                             // all four warps leave together
            ++k;
            if (lane == 0) mbar_arrive(b_box_empty);                    // the epilogue may announce its next segment
            const size_t blk = (size_t)slot * nrt + rb;
            if (sg.nu != upi) {
                // this cluster reduced only some of the row block's column tiles: the last to arrive finishes
                __threadfence();
                asm volatile("bar.sync 4, 128;" ::: "memory");
                if (row == 0) arrival = atomicAdd(&P.tc_cnt[blk], (unsigned)sg.nu);
                asm volatile("bar.sync 4, 128;" ::: "memory");
                const unsigned before = arrival;
                asm volatile("bar.sync 4, 128;" ::: "memory");          // `arrival` is free again
                if ((int)before + sg.nu != upi) continue;
                if (row == 0) P.tc_cnt[blk] = 0u;
                __threadfence();
            }
            float m = NEG_BIG;
            double sm = 0.0;
            for (int f = 0; f < 2 * upi; ++f) {                         // units in order, even chunks before odd ones
                const size_t q = (blk * (2 * TC_MAX_SPLIT) + f) * TC_BM + row;
                const float mo = reinterpret_cast<volatile float *>(P.tc_pm)[q];
                const double so = reinterpret_cast<volatile double *>(P.tc_ps)[q];
                const float mn = fmaxf(m, mo);
                sm = sm * (double)pow2i(m - mn) + so * (double)pow2i(mo - mn);
                m = mn;
            }
            const bool frozen = (P.mode == MODE_MASKED) && P.state[slot] != 0;
            const int i = rb * TC_BM + row;
            unsigned long long term = 0ull;
            if (i < nrows) {
                const double tr = finish_one_row<float>(P, c, leg, slot, (int)FORM_DOT, i, m, sm, 0.f, !frozen && leg != LEG_V && !P.dry_run);
                if (leg != LEG_G) term = residual_fixed(P, leg, slot, tr, frozen);
            }
            if (leg != LEG_G) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) term += __shfl_down_sync(0xffffffffu, term, off);
                if (lane == 0) red[fw] = term;
                asm volatile("bar.sync 4, 128;" ::: "memory");
                if (row == 0 && !P.dry_run) finish_lane_residual(P, leg, slot, ((red[0] + red[1]) + red[2]) + red[3]);
                asm volatile("bar.sync 4, 128;" ::: "memory");          // red[] is free again
            }
        }
    } else {
        // ---------------- epilogue: thread e <-> row (e & 127) of this CTA's block <-> TMEM lane (e & 127);
        // warps 0-3 take the even 32-column chunks of every tile, warps 4-7 the odd ones
        const int e = tid, half = warp >> 2, row = e & 127;
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = true;
        int tg = 0, nbox = 0;
        while (ok && it.next(sg)) {
            if (TC2_SKIP(sg.slot)) continue;
            const int slot = sg.slot, rb = 2 * sg.pb + (int)rank;
            const bool ghost = rb >= nrt;
            const float *colt = rows_x ? reinterpret_cast<const float *>(P.gt) + (size_t)slot * cp
                                       : reinterpret_cast<const float *>(P.ft[c.parity]) + (size_t)slot * cp;
            const float two_s = (float)(2.0 * P.scale[slot]);
            float mx = NEG_BIG, ts = 0.f;
            double sd = 0.0;
            float g_next = (sg.t0 * TC2_BN + e < cp) ? colt[sg.t0 * TC2_BN + e] : NEG_BIG;   // column term, one tile ahead
            for (int t = sg.t0; t < sg.t1; ++t, ++tg) {
                const int buf = tg & 1;
#ifdef SKB_TC_DEBUG
                const long long tb0 = clock64();
#endif
                asm volatile("bar.sync 1, 256;" ::: "memory");          // everyone is done with the previous tile's column terms
#ifdef SKB_TC_DEBUG
                dbg_w1 += clock64() - tb0;
#endif
                gts[e] = g_next;
                {
                    const int j = (t + 1) * TC2_BN + e;
                    g_next = (t + 1 < sg.t1 && j < cp) ? colt[j] : NEG_BIG;
                }
                ok = TC_TIMED_WAIT(dbg_w0, mbar_wait(b_tfull + 8 * buf, (tg >> 1) & 1, ab));
#ifdef SKB_TC_DEBUG
                const long long tb1 = clock64();
#endif
                ok = epi_all(ok);                                       // also publishes the column terms
#ifdef SKB_TC_DEBUG
                dbg_w1 += clock64() - tb1;
#endif
                if (!ok) break;
                tc_fence_after();
                tc_reduce_tile<TC2_BN>(lane_base + (uint32_t)(buf * TC2_BN), gts, half, two_s, mx, ts, sd);
                sd += (double)ts;
                ts = 0.f;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {                                        // one arrival per warp: this accumulator is read
                    if (leader) mbar_arrive(b_tempty + 8 * buf);
                    else mbar_arrive_remote(b_tempty_leader + 8 * buf);
                }
                if ((t + 1) % g == 0 || t + 1 == ntiles) {
                    // a unit is complete: its row results go to scratch and the reduction starts afresh
                    if (!ghost) {
                        const size_t q = ((((size_t)slot * nrt + rb) * TC_MAX_SPLIT + t / g) * 2 + half) * TC_BM + row;
                        P.tc_pm[q] = mx;
                        P.tc_ps[q] = sd;
                    }
                    mx = NEG_BIG;
                    sd = 0.0;
                }
            }
            if (!ok) break;
            // tell the filing warps that this segment's units are in scratch (at most one announcement ahead)
            if (!ghost && nbox > 0) mbar_wait(b_box_empty, (nbox - 1) & 1, ab);
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (e == 0 && !ghost) mbar_arrive(b_box_full);
            if (!ghost) ++nbox;
        }
    }
#undef TC2_SKIP
    if (abort_flag) {
        // a wait ran out: give copies that may still be in flight time to land in this CTA's
        // shared memory before it is released (bounded: ~0.1 ms)
        const long long t0 = clock64();
        while (clock64() - t0 < 200000LL) { }
    }
#ifdef SKB_TC_DEBUG
    if (blockIdx.x < 2 && leg == LEG_F && (lane == 0) && (warp == 0 || warp == 4 || warp >= TC_EPI_WARPS))
        printf("[tc2 dbg] rank %u warp %d: total %lld clk, wait0 %lld, wait1 %lld (producer: empty; mma: full, tmem-empty; epilogue: tmem-full) tiles %d chunks/tile %d stages %d units %d clusters %d\n",
               rank, warp, clock64() - dbg_t0, dbg_w0, dbg_w1, ntiles, nkc, nstages, U, ncl);
#endif
    tc_fence_before();
    __syncthreads();
    cluster_barrier();                                  // the pair is done with each other's memory
    tc_fence_after();
    if (warp == TC_EPI_WARPS + 1) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    if (abort_flag) {
        if (tid == 0) atomicOr(&P.ctl->error, ERR_WAIT);
    }
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing will ever complete
// and must come back with `false` once its clock budget is spent.
__global__ void wait_probe_kernel(int *out, long long budget)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const long long t0 = clock64();
        const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, budget);
        out[0] = ok ? 0 : 1;                       // 1: the wait gave up
        out[1] = abort_flag;
        out[2] = (int)((clock64() - t0) >> 10);    // kilo-clocks spent
    }
}

void launch_wait_probe(int *out, long long budget_clocks, cudaStream_t st)
{
    wait_probe_kernel<<<1, 32, 0, st>>>(out, budget_clocks);
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool tc_eligible(int d, bool bf16) { return bf16 && d >= 64 && d <= 512 && d % 64 == 0; }

// d <= 256: 128-column tiles and two ring stages, small enough for two CTAs per SM (the second
// CTA's MMAs cover this CTA's prologue and epilogue).  d > 256: the persistent CTA-pair kernel
// (its ring needs two stages and no more than d/64).
constexpr size_t TC_SMEM_LIMIT = 232448;                  // 227 KB: static + dynamic shared memory of one CTA
static bool tc_wide(int d) { return d > 256; }             // measured: the two kernels break even at d = 256
size_t tc_smem_bytes(int d) { return (size_t)(d / TC_BK + 2) * TC_CHUNK; }   // the two-CTAs-per-SM kernel

// Tensor map of one tiled operand copy: rows of 64 bf16 (128 B, contiguous), 128-row boxes.
const char *tc_make_map(void *out_map, void *base, int W, int npts, int d)
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || !p)
            return "cuTensorMapEncodeTiled is not available";
        fn = (EncodeTiledFn)p;
    }
    const cuuint64_t rows = (cuuint64_t)W * ((npts + TC_BM - 1) / TC_BM) * (d / TC_BK) * TC_BM;
    const cuuint64_t gdim[2] = {(cuuint64_t)TC_BK, rows};
    const cuuint64_t gstr[1] = {(cuuint64_t)TC_BK * 2};
    const cuuint32_t box[2] = {TC_BK, TC_BM};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn((CUtensorMap *)out_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, gdim, gstr, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? nullptr : "cuTensorMapEncodeTiled failed";
}

size_t tc_tiled_bytes(int W, int npts, int d) { return (size_t)W * ((npts + TC_BM - 1) / TC_BM) * (d / TC_BK) * TC_CHUNK; }

// Copies [W][npts][d] bf16 into the tiled layout [W][tile][chunk][128][64]; points past npts become zeros.
__global__ void __launch_bounds__(256) retile_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int npts, int d)
{
    const int nkc = d / TC_BK, ntile = (npts + TC_BM - 1) / TC_BM;
    const int blk = blockIdx.x, tile = blk / nkc, kc = blk % nkc, slot = blockIdx.y;
    uint4 *out = dst + ((size_t)(slot * ntile + tile) * nkc + kc) * (TC_CHUNK / 16);
    for (int q = threadIdx.x; q < TC_BM * 8; q += 256) {
        const int r = q >> 3, c = q & 7, pt = tile * TC_BM + r;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (pt < npts) v = src[((size_t)(slot * (size_t)npts + pt) * d + kc * TC_BK) / 8 + c];
        out[q] = v;
    }
}

void launch_retile(const void *src, void *dst, int W, int npts, int d, cudaStream_t st)
{
    dim3 grid(((npts + TC_BM - 1) / TC_BM) * (d / TC_BK), W);
    retile_kernel<<<grid, 256, 0, st>>>((const uint4 *)src, (uint4 *)dst, npts, d);
}

void launch_update_tc(const Dev &P, const void *maps, int leg, int width, cudaStream_t st)
{
    // dynamic shared memory: the tiles, plus what it takes to start them on a 1024-byte boundary
    static size_t pad[2] = {0, 0};
    static size_t pair_static = 0;
    static int sm_count = 0;
    static bool attr_set = false;
    if (!attr_set) {
        cudaFuncAttributes fa;
        cudaFuncGetAttributes(&fa, update_tc_kernel<2, 128>);
        pad[0] = (1024 - fa.sharedSizeBytes % 1024) % 1024;
        cudaFuncGetAttributes(&fa, update_tc_pair_kernel);
        pad[1] = (1024 - fa.sharedSizeBytes % 1024) % 1024;
        pair_static = fa.sharedSizeBytes;
        cudaFuncSetAttribute(update_tc_kernel<2, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(tc_smem_bytes(256) + pad[0]));
        cudaFuncSetAttribute(update_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(TC_SMEM_LIMIT - pair_static));
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
        attr_set = true;
    }
    const CUtensorMap *tm = reinterpret_cast<const CUtensorMap *>(maps);
    const int nrows = (leg == LEG_F) ? P.n : P.m, ncols = (leg == LEG_F) ? P.m : P.n;
    const int nrt = (nrows + TC_BM - 1) / TC_BM;
    const int lanes = width < 1 ? 1 : width;
    if (!tc_wide(P.d)) {
        launch_pdl(update_tc_kernel<2, 128>, dim3(nrt, lanes), dim3(TC_THREADS), tc_smem_bytes(P.d) + pad[0], st, tm[0], tm[1], P, leg);
        return;
    }
    // as many 16 KB ring stages as fit beside the resident row block (six at d = 512), at least
    // two and no more than a tile has chunks (see the kernel's header)
    const int nkc = P.d / TC_BK;
    const size_t room = TC_SMEM_LIMIT - pair_static - pad[1] - (size_t)nkc * TC_CHUNK;
    int nst = (int)(room / TC_CHUNK);
    if (nst > TC2_MAX_STAGES) nst = TC2_MAX_STAGES;
    if (nst > nkc) nst = nkc;
    // one cluster per SM pair, fewer if there are fewer units of work
    const int ntl = (ncols + TC2_BN - 1) / TC2_BN, g = tc_unit_tiles(ntl);
    const long long units = (long long)lanes * ((nrt + 1) / 2) * ((ntl + g - 1) / g);
    const int ncl = units < sm_count / 2 ? (int)units : sm_count / 2;
    launch_pdl(update_tc_pair_kernel, dim3(2 * ncl), dim3(TC2_THREADS), (size_t)(nkc + nst) * TC_CHUNK + pad[1], st, tm[0], tm[1], P, leg, nst);
}

}  // namespace skb
