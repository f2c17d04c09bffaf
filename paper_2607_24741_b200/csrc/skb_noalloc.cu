// Allocation-free row-residual check.
//
// Some callers of this library may not allocate device memory at all: a host application
// that gives every component a fixed memory budget at start-up and forbids later driver
// allocations, or a latency-critical loop that cannot afford the implicit device-wide
// synchronisation of cudaMalloc / cudaFree.  The batch API already takes its workspace from
// the caller, but a caller who only wants to audit a plan it already holds (potentials from
// an earlier solve, a warm start, another solver) would still have to size and provide
// that workspace.  This entry point needs none: the per-CTA partial sums and the arrival
// counters of the fused residual reduction live in a fixed array that is part of the
// library image, so every GPU that loads the library carries SKB_STATIC_SCRATCH_BYTES of it
// until the process exits.
//
// It is the row screen of the update kernel in its plainest form: for every lane
//     r_row = sum_i | sum_j exp((f_i + g_j - |x_i - y_j|^2) / eps) - a_i |,
// float64 arithmetic, one thread per row, per-CTA partial sums combined in a fixed order by
// the last CTA of the lane to arrive.
#include <cuda_runtime.h>
#include <mutex>
#include <string>

#include "../../include/sinkhorn_batch.h"

namespace {

constexpr int NA_THREADS = 128;                       // rows per CTA
constexpr int NA_MAX_LANES = SKB_STATIC_MAX_LANES;    // 256
constexpr int NA_MAX_BLOCKS = SKB_STATIC_MAX_ROWS / NA_THREADS;   // 64 row blocks per lane
constexpr int NA_MAX_DEVICES = 64;

struct Scratch {
    double partial[NA_MAX_LANES][NA_MAX_BLOCKS];      // per-CTA L1 partial sums
    unsigned arrived[NA_MAX_LANES];                   // CTAs of the lane that have finished
};
static_assert(sizeof(Scratch) <= SKB_STATIC_SCRATCH_BYTES, "scratch larger than documented");

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress;
// it is not a device address and must never be handed to a kernel directly.
static __device__ __align__(256) unsigned char g_scratch[SKB_STATIC_SCRATCH_BYTES];

std::mutex g_mu;
Scratch *g_dev_scratch[NA_MAX_DEVICES] = {};
thread_local std::string g_err;       // text of the calling thread's last failure; empty after a success

__global__ void __launch_bounds__(NA_THREADS) row_residual_kernel(
    Scratch *sc, const float *x, const float *y, const float *a, const double *f, const double *g,
    const float *eps, int n, int m, int d, float *r_row)
{
    __shared__ double red[NA_THREADS / 32];
    __shared__ int is_last;
    const int lane_id = blockIdx.y, tid = threadIdx.x;
    const int i = blockIdx.x * NA_THREADS + tid;
    const double inv_eps = 1.0 / (double)eps[lane_id];
    const float *xl = x + (size_t)lane_id * n * d, *yl = y + (size_t)lane_id * m * d;
    const double *fl = f + (size_t)lane_id * n, *gl = g + (size_t)lane_id * m;
    double term = 0.0;
    if (i < n) {
        double mx = -1.0e300, s = 0.0;
        for (int j = 0; j < m; ++j) {
            double c = 0.0;
            for (int k = 0; k < d; ++k) {
                const double t = (double)xl[(size_t)i * d + k] - (double)yl[(size_t)j * d + k];
                c += t * t;
            }
            const double v = (fl[i] + gl[j] - c) * inv_eps;
            if (v > mx) { s *= exp(mx - v); mx = v; }
            s += exp(v - mx);
        }
        term = fabs(exp(mx) * s - (double)a[(size_t)lane_id * n + i]);
    }
    for (int off = 16; off > 0; off >>= 1) term += __shfl_down_sync(0xffffffffu, term, off);
    if ((tid & 31) == 0) red[tid >> 5] = term;
    __syncthreads();
    if (tid == 0) {
        double p = 0.0;
        for (int w = 0; w < NA_THREADS / 32; ++w) p += red[w];
        sc->partial[lane_id][blockIdx.x] = p;
        __threadfence();
        is_last = (atomicAdd(&sc->arrived[lane_id], 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last || tid != 0) return;
    __threadfence();
    double tot = 0.0;
    for (unsigned b = 0; b < gridDim.x; ++b) tot += reinterpret_cast<volatile double *>(sc->partial[lane_id])[b];
    sc->arrived[lane_id] = 0u;              // leave the counter ready for the next call
    r_row[lane_id] = (float)tot;
}

skb_status fail(skb_status st, const std::string &msg)
{
    g_err = msg;
    return st;
}

}  // namespace

extern "C" const char *sinkhorn_row_residual_static_last_error(void) { return g_err.c_str(); }

extern "C" skb_status sinkhorn_row_residual_static(const float *x, const float *y, const float *a,
                                                   const double *f, const double *g, const float *eps,
                                                   int W, int n, int m, int d, float *r_row, void *stream)
{
    std::lock_guard<std::mutex> lock(g_mu);
    if (!x || !y || !a || !f || !g || !eps || !r_row) return fail(SKB_ERR_NULL, "all data pointers are required");
    if (W < 1 || n < 1 || m < 1 || d < 1) return fail(SKB_ERR_SHAPE, "W, n, m, d must be >= 1");
    if (W > SKB_STATIC_MAX_LANES || n > SKB_STATIC_MAX_ROWS)
        return fail(SKB_ERR_SHAPE, "beyond the static scratch: at most " + std::to_string(SKB_STATIC_MAX_LANES) +
                                       " lanes and " + std::to_string(SKB_STATIC_MAX_ROWS) + " source points per lane");
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(SKB_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    if (dev < 0 || dev >= NA_MAX_DEVICES) return fail(SKB_ERR_STATE, "device ordinal out of range");
    if (!g_dev_scratch[dev]) {
        // first call on this device: resolve the device address of the static array
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_scratch);
        if (e != cudaSuccess) return fail(SKB_ERR_CUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
        g_dev_scratch[dev] = reinterpret_cast<Scratch *>(p);
    }
    Scratch *sc = g_dev_scratch[dev];
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the arrival counters must start at zero
    e = cudaMemsetAsync(sc->arrived, 0, sizeof(sc->arrived), st);
    if (e != cudaSuccess) return fail(SKB_ERR_CUDA, std::string("cudaMemsetAsync: ") + cudaGetErrorString(e));
    dim3 grid((n + NA_THREADS - 1) / NA_THREADS, W);
    row_residual_kernel<<<grid, NA_THREADS, 0, st>>>(sc, x, y, a, f, g, eps, n, m, d, r_row);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(SKB_ERR_CUDA, std::string("launch: ") + cudaGetErrorString(e));
    g_err.clear();
    return SKB_OK;
}
