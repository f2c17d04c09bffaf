// Self-test family: measured issue rates of the arithmetic units the update kernels are bound
// by, so that a roofline fraction can be quoted against what the machine delivers and not only
// against the nominal unit counts.  Each kernel is a loop of independent dependency chains of
// one instruction kind in registers (no memory traffic), timed with CUDA events.
#include <string>

#include "../../include/sinkhorn_batch.h"
#include "skb_host.h"

namespace skb {

constexpr int UR_THREADS = 256;
constexpr int UR_CHAINS = 8;        // independent chains per thread: enough to cover the pipe latency
constexpr int UR_ITERS = 4096;       // a multiple of UR_UNROLL
constexpr int UR_UNROLL = 8;         // chain steps per loop trip, so that the loop's own instructions are a few percent
constexpr int UR_CTAS_PER_SM = 8;

// kind 0: fma.rn.f32, 1: fma.rn.f32x2 (two FMAs per instruction), 2: fma.rn.f64, 3: ex2.approx.ftz.f32
template <int KIND>
__global__ void __launch_bounds__(UR_THREADS) unit_rate_kernel(float *sink, const float seed)
{
    const float t = seed + 1e-9f * (float)threadIdx.x;
    if constexpr (KIND == 0) {
        float a[UR_CHAINS];
#pragma unroll
        for (int c = 0; c < UR_CHAINS; ++c) a[c] = t + (float)c;
#pragma unroll 1
        for (int i = 0; i < UR_ITERS / UR_UNROLL; ++i) {
#pragma unroll
            for (int u = 0; u < UR_UNROLL; ++u)
#pragma unroll
                for (int c = 0; c < UR_CHAINS; ++c) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(a[c]) : "f"(0.999f), "f"(t));
        }
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < UR_CHAINS; ++c) s += a[c];
        if (s == 123.456f) sink[0] = s;
    } else if constexpr (KIND == 1) {
        unsigned long long a[UR_CHAINS], m, b;
        asm("mov.b64 %0, {%1, %1};" : "=l"(m) : "f"(0.999f));
        asm("mov.b64 %0, {%1, %1};" : "=l"(b) : "f"(t));
#pragma unroll
        for (int c = 0; c < UR_CHAINS; ++c) asm("mov.b64 %0, {%1, %1};" : "=l"(a[c]) : "f"(t + (float)c));
#pragma unroll 1
        for (int i = 0; i < UR_ITERS / UR_UNROLL; ++i) {
#pragma unroll
            for (int u = 0; u < UR_UNROLL; ++u)
#pragma unroll
                for (int c = 0; c < UR_CHAINS; ++c) asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(a[c]) : "l"(m), "l"(b));
        }
        unsigned long long s = 0ull;
#pragma unroll
        for (int c = 0; c < UR_CHAINS; ++c) s ^= a[c];
        if (s == 0x123456789abcdefull) sink[0] = 1.f;
    } else if constexpr (KIND == 2) {
        double a[UR_CHAINS];
        const double td = (double)t;
#pragma unroll
        for (int c = 0; c < UR_CHAINS; ++c) a[c] = td + (double)c;
#pragma unroll 1
        for (int i = 0; i < UR_ITERS / UR_UNROLL; ++i) {
#pragma unroll
            for (int u = 0; u < UR_UNROLL; ++u)
#pragma unroll
                for (int c = 0; c < UR_CHAINS; ++c) asm volatile("fma.rn.f64 %0, %0, %1, %2;" : "+d"(a[c]) : "d"(0.999), "d"(td));
        }
        double s = 0.0;
#pragma unroll
        for (int c = 0; c < UR_CHAINS; ++c) s += a[c];
        if (s == 123.456) sink[0] = (float)s;
    } else {
        float a[UR_CHAINS];
#pragma unroll
        for (int c = 0; c < UR_CHAINS; ++c) a[c] = t + 0.01f * (float)c;
#pragma unroll 1
        for (int i = 0; i < UR_ITERS / UR_UNROLL; ++i) {
#pragma unroll
            for (int u = 0; u < UR_UNROLL; ++u)
#pragma unroll
                for (int c = 0; c < UR_CHAINS; ++c)      // a <- 2^(-a): stays in (0.5, 1), no overflow, no flush
                    asm volatile("{ .reg .f32 t; neg.f32 t, %0; ex2.approx.ftz.f32 %0, t; }" : "+f"(a[c]));
        }
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < UR_CHAINS; ++c) s += a[c];
        if (s == 123.456f) sink[0] = s;
    }
}

}  // namespace skb

using namespace skb;

extern "C" skb_status sinkhorn_batch_selftest_unit_rates(double *ops_per_second, float *sink, void *stream)
{
    if (!ops_per_second || !sink) return SKB_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SKB_ERR_CUDA;
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess) return SKB_ERR_CUDA;
    if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return SKB_ERR_CUDA; }
    const dim3 grid(sms * UR_CTAS_PER_SM), block(UR_THREADS);
    const double per_launch = (double)grid.x * UR_THREADS * UR_CHAINS * UR_ITERS;
    const double ops_per_instr[4] = {1.0, 2.0, 1.0, 1.0};
    cudaError_t e = cudaSuccess;
    for (int kind = 0; kind < 4 && e == cudaSuccess; ++kind) {
        float best = 0.f;
        for (int rep = 0; rep < 4; ++rep) {                        // first repetition warms up
            cudaEventRecord(a, st);
            switch (kind) {
            case 0: unit_rate_kernel<0><<<grid, block, 0, st>>>(sink, 0.5f); break;
            case 1: unit_rate_kernel<1><<<grid, block, 0, st>>>(sink, 0.5f); break;
            case 2: unit_rate_kernel<2><<<grid, block, 0, st>>>(sink, 0.5f); break;
            default: unit_rate_kernel<3><<<grid, block, 0, st>>>(sink, 0.5f); break;
            }
            cudaEventRecord(b, st);
            if ((e = cudaEventSynchronize(b)) != cudaSuccess) break;
            float ms = 0.f;
            if ((e = cudaEventElapsedTime(&ms, a, b)) != cudaSuccess) break;
            if (rep > 0 && (best == 0.f || ms < best)) best = ms;
        }
        ops_per_second[kind] = best > 0.f ? per_launch * ops_per_instr[kind] / ((double)best * 1e-3) : 0.0;
    }
    cudaEventDestroy(a); cudaEventDestroy(b);
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : SKB_ERR_CUDA;
}
