// Tensor-core variant of the update kernel for bf16 point clouds with a deep cross term
// (d a multiple of 64, 64 <= d <= 512): the only place on the path that is a dense
// contraction.
//
// For a block of 128 row points the CTA computes S = R . C^T against column tiles of 128
// points with tcgen05.mma (bf16 operands straight from the caller's layout, fp32
// accumulators in tensor memory), then log2 pi_ij = 2 s S_ij + ct_j and the same online
// max / sum-of-exp2 reduction and float64 epilogue as the SIMT kernels (dot form).
//
// Warp roles (192 threads):
//   warps 0-3  epilogue: thread e owns row e = TMEM lane e; tcgen05.ld 32 columns at a time,
//              fma with the column term, online logsumexp entirely in registers (no shuffles)
//   warp 4     producer: one lane issues TMA loads of pre-tiled operand copies (every
//              128-point x 64-dimension chunk is one contiguous 16 KB block in the workspace,
//              which TMA streams at about twice the rate of 1 KB-strided rows; 128-byte
//              swizzle; points past the end are stored as zeros): the row block once
//              (d/64 chunks of 16 KB, riding on the first tile's barriers), and column
//              chunks through a ring of 2 (d <= 256, 128-column tiles, two CTAs per SM) or
//              3 stages (d > 256, 256-column tiles of two chunks each)
//   warp 5     allocates the TMEM columns of two accumulators (2 x 128 or 2 x 256); one lane issues
//              the MMAs (4 x K=16 per 64-wide chunk) and commits to the ring's empty barriers and
//              to the accumulator-full barrier, so the next tile's MMAs overlap this tile's
//              exponentials.
// Every mbarrier wait is bounded by a clock budget; on expiry the kernel raises ERR_WAIT in
// the control block, all roles leave their loops, tensor memory is freed and the kernel
// returns (the host reports SKB_ERR_CUDA).
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdio>

#include "skb_update.cuh"
#include "skb_host.h"

namespace skb {

constexpr int TC_THREADS = 192;
constexpr int TC_MAX_STAGES = 4;
constexpr int TC_BM = 128, TC_BK = 64;
constexpr uint32_t TC_CHUNK = TC_BM * TC_BK * 2;          // 16 KB: 128 points x 64 bf16
constexpr long long TC_WAIT_CLOCKS = 2000000000LL;        // ~1 s
__device__ long long g_wait_clocks = TC_WAIT_CLOCKS;      // budget of every bounded wait (a self-test shortens it)

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
__device__ __forceinline__ bool mbar_wait(uint32_t a, uint32_t parity, volatile int *abort_flag)
{
    const long long t0 = clock64();
    while (!mbar_try_wait(a, parity)) {
        if (*abort_flag) return false;
        if (clock64() - t0 > g_wait_clocks) { *abort_flag = 1; return false; }
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
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
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
__global__ void __launch_bounds__(TC_THREADS, 1)
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
    __shared__ int is_last;

    pdl_enter();
    const Ctl c = *P.ctl;
    if (c.done) return;
    const int slot = blockIdx.y;
    if (slot >= c.n_phys) return;
    if (leg != LEG_V && c.static_final) return;
    if (leg == LEG_V && !(c.static_final || P.flag[slot])) return;
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
        for (int b = 0; b < 2; ++b) { mbar_init(b_tfull + 8 * b, 1); mbar_init(b_tempty + 8 * b, 128); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        if (TC_BN == 256) asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&tmem_holder)) : "memory");
        else asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&tmem_holder)) : "memory");
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

    if (warp == 4) {
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
    } else if (warp == 5) {
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
        // ---------------- epilogue: thread e <-> row e <-> TMEM lane e
        const int e = tid;
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        bool ok = true;
        for (int t = 0; t < ntiles && ok; ++t) {
            const int buf = t & 1;
#pragma unroll
            for (int h = 0; h < TC_BN / 128; ++h) {
                const int j = t * TC_BN + h * 128 + e;
                gts[buf][h * 128 + e] = (j < cp) ? colt[j] : NEG_BIG;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            ok = TC_TIMED_WAIT(dbg_w0, mbar_wait(b_tfull + 8 * buf, (t >> 1) & 1, ab));
            if (!ok) break;
            tc_fence_after();
            float ts = 0.f;
#pragma unroll 1
            for (int cb = 0; cb < TC_BN; cb += 32) {
                float v[32];
                tc_ld32(lane_base + (uint32_t)(buf * TC_BN + cb), v);
                float mt = NEG_BIG;
#pragma unroll
                for (int q = 0; q < 32; ++q) {
                    v[q] = fmaf(v[q], two_s, gts[buf][cb + q]);
                    mt = fmaxf(mt, v[q]);
                }
                if (mt > mx + 8.0f) {
                    const float mn = ceilf(mt);
                    const float fac = pow2i(mx - mn);
                    ts *= fac;
                    sd *= (double)fac;
                    mx = mn;
                }
#pragma unroll
                for (int q = 0; q < 32; ++q) ts += ex2_fast(v[q] - mx);
            }
            sd += (double)ts;
            tc_fence_before();
            mbar_arrive(b_tempty + 8 * buf);                // all 128 rows have read this accumulator
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");     // every row is done with the column terms
        row_m[e] = mx;
        row_s[e] = ok ? sd : __longlong_as_double(0x7ff8000000000000LL);
        row_h[e] = 0.f;
    }
    if (abort_flag) {
        // a wait ran out: give copies that may still be in flight time to land in this CTA's
        // shared memory before it is released (bounded: ~0.1 ms)
        const long long t0 = clock64();
        while (clock64() - t0 < 200000LL) { }
    }
#ifdef SKB_TC_DEBUG
    if (blockIdx.x == 1 && blockIdx.y == 3 && leg == LEG_F && (lane == 0) && (warp == 0 || warp >= 4))
        printf("[tc dbg] warp %d: total %lld clk, wait0 %lld, wait1 %lld (producer: empty; mma: full, tmem-empty; epilogue: tmem-full) tiles %d chunks/tile %d\n",
               warp, clock64() - dbg_t0, dbg_w0, dbg_w1, ntiles, nkc);
#endif
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 5) {
        if (TC_BN == 256) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
    }
    if (abort_flag) {
        if (tid == 0) atomicOr(&P.ctl->error, ERR_WAIT);
    }
    finish_rows<float, TC_BM, TC_THREADS>(P, c, leg, slot, (int)FORM_DOT, row_m, row_s, row_h, red, &is_last);
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
        const long long saved = g_wait_clocks;
        g_wait_clocks = budget;
        const long long t0 = clock64();
        const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag);
        out[0] = ok ? 0 : 1;                       // 1: the wait gave up
        out[1] = abort_flag;
        out[2] = (int)((clock64() - t0) >> 10);    // kilo-clocks spent
        g_wait_clocks = saved;
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

// two ring stages when that lets two CTAs share an SM (d <= 256: the second CTA's MMAs cover
// this CTA's prologue and epilogue), four otherwise
// beyond d = 256 the row block lives in tensor memory, which leaves shared memory to a 12-stage ring
// d <= 256: 128-column tiles, two ring stages, small enough for two CTAs per SM (the second CTA's MMAs
// cover this CTA's prologue and epilogue).  d > 256: 256-column tiles (the tensor pipe runs 128x256 MMAs
// about twice as efficiently as 128x128 ones), three 32 KB stages beside the 128 KB row block.
static bool tc_wide(int d) { return d > 256; }
size_t tc_smem_bytes(int d) { return (size_t)(d / TC_BK + (tc_wide(d) ? 6 : 2)) * TC_CHUNK; }

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
    static bool attr_set = false;
    if (!attr_set) {
        cudaFuncAttributes fa;
        cudaFuncGetAttributes(&fa, update_tc_kernel<2, 128>);
        pad[0] = (1024 - fa.sharedSizeBytes % 1024) % 1024;
        cudaFuncGetAttributes(&fa, update_tc_kernel<3, 256>);
        pad[1] = (1024 - fa.sharedSizeBytes % 1024) % 1024;
        cudaFuncSetAttribute(update_tc_kernel<2, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(tc_smem_bytes(256) + pad[0]));
        cudaFuncSetAttribute(update_tc_kernel<3, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(tc_smem_bytes(512) + pad[1]));
        attr_set = true;
    }
    const CUtensorMap *tm = reinterpret_cast<const CUtensorMap *>(maps);
    const int nrows = (leg == LEG_F) ? P.n : P.m;
    dim3 grid((nrows + TC_BM - 1) / TC_BM, width < 1 ? 1 : width);
    if (!tc_wide(P.d)) launch_pdl(update_tc_kernel<2, 128>, grid, dim3(TC_THREADS), tc_smem_bytes(P.d) + pad[0], st, tm[0], tm[1], P, leg);
    else launch_pdl(update_tc_kernel<3, 256>, grid, dim3(TC_THREADS), tc_smem_bytes(P.d) + pad[1], st, tm[0], tm[1], P, leg);
}

}  // namespace skb
