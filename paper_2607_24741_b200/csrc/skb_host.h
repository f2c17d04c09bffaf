// Host-side declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include "skb_device.cuh"

namespace skb {

// Launch with programmatic stream serialization allowed (the kernel must call pdl_enter()).
//
// Invariants the kernels of a cycle rely on (f-leg, column check, plan, emit/move, g-leg, in that
// order on one stream):
//  - every kernel executes griddepcontrol.wait in at least one block before it completes, so that
//    "my predecessor has completed" implies "everything earlier in the stream has completed";
//  - the control block is written by the plan kernel only, coordinates and the per-slot scalars by
//    the plan and emit/move kernels only;
//  - a kernel that reads state BEFORE its own wait (the SIMT f-leg: control block, row coordinates,
//    row potentials; the column check: control block) may do so because the kernel that released it
//    is a g-leg (of this batch or of another batch sharing the stream), and g-legs release their
//    dependents only after their own wait: by then the plan and emit/move kernels before it are
//    complete, and nothing between them and the early reader writes what it reads early;
//  - kernels launched without the attribute (set-up, read-back, a caller's own kernels) neither
//    start early nor release early, so they may sit anywhere in the stream.
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Update-kernel variant: compute type, padded dimension, rows per thread, column split.
struct Variant {
    int f64, xf, DP, R, CS;   // xf: float64 arguments with fp32 special-function exponentials
    int rows_per_cta;
    size_t smem;
    int (*launch)(const Dev &, int leg, int width, cudaStream_t);   // 1: the guard band's pool rode in a column-check launch
    // several whole cycles per launch, one thread-block cluster per lane; null where there is none
    void (*launch_cycles)(const Dev &, int cycles, int width, cudaStream_t);
    // does a lane of n x m points fit the shared-memory-resident version of the multi-cycle kernel?
    bool (*lane_fits_shared)(int n, int m);
};
constexpr int MAX_CLUSTER_BLOCKS = MAX_CLUSTER_RANKS;   // a lane needs at most this many row blocks
constexpr int MAX_CYCLES_IN_LAUNCH = 64;    // upper bound on the cycles one multi-cycle launch runs
// Picks the variant for a shape (depends on the static shape only, so that every mode
// and every run of the same batch uses the same reduction order).  Null if unsupported.
const Variant *choose_variant(int W, int n, int m, int d, bool f64, bool fast_exp, int force_cs);
int padded_dim(int d);

void launch_lane_stats(const Dev &P, const void *x, const void *y, const float *eps, int slot0, int lane0, int count,
                       int cycle0, cudaStream_t st);
void launch_prep(const Dev &P, const void *x, const void *y, const float *a, const float *b, int slot0, int count, cudaStream_t st);
void launch_refill_ctl(const Dev &P, int count, cudaStream_t st);
void launch_warm(const Dev &P, const double *f0, const double *g0, cudaStream_t st);
int launch_plan(const Dev &P, int width, cudaStream_t st);        // both return the number of kernels launched
// tensor-core update kernel (bf16 inputs, d a multiple of 64 up to 512)
bool tc_eligible(int d, bool bf16);
const char *tc_make_map(void *out_map, void *base, int W, int npts, int d);
size_t tc_tiled_bytes(int W, int npts, int d);
void launch_retile(const void *src, void *dst, int W, int npts, int d, cudaStream_t st);
void launch_wait_probe(int *out, long long budget_clocks, cudaStream_t st);
void launch_guard_pool(const Dev &P, cudaStream_t st);
void launch_guard_strips(void *base, const GuardList &gl, bool fill, int *bad, cudaStream_t st);
void launch_update_tc(const Dev &P, const void *maps, int leg, int width, cudaStream_t st);
int launch_emit_move(const Dev &P, int width, cudaStream_t st);
int launch_plan_cycles(const Dev &P, int width, int cycles, cudaStream_t st);
void launch_gather(const Dev &P, void *f, void *g, bool f64, cudaStream_t st);
void launch_gather_audit(const Dev &P, float *rrow, float *rcol, int *flagged, cudaStream_t st);
void launch_apply_plan(const Dev &P, const void *x, const void *y, const float *eps, const float *v, int dv, float *out,
                       int lanes, cudaStream_t st);
void launch_gather_small(const Dev &P, int *depth, int *status, float *rrow, float *rcol, cudaStream_t st);

}  // namespace skb
