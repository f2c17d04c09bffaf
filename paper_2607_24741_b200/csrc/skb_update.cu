// Instantiations of the streaming update kernel and the shape -> variant choice.
#include <cstdlib>
#include "skb_update.cuh"
#include "skb_update_bigd.cuh"
#include "skb_host.h"

namespace skb {

constexpr size_t RESIDENT_SMEM_LIMIT = 52 * 1024; // shared memory of a block of the resident multi-cycle kernel: four blocks fit an SM

constexpr long long NARROW_BLOCKS = 148 * 4;      // below this many blocks some SM has fewer than four

// Grid rows (of `per_row` blocks each) that hold the guard band's pool of about two blocks per SM.
// None when the launch has no room for them (grid.y is 16 bits): the caller then runs the pool as
// a launch of its own.
static int pool_rows(int per_row, bool on, int lanes)
{
    const int rows = on ? (2 * 148 + per_row - 1) / per_row : 0;
    return lanes + rows <= 65535 ? rows : 0;
}

template <typename T, int DP, int CS, int XF>
static int launch_update(const Dev &P, int leg, int width, cudaStream_t st)   // returns 1 if the guard band's pool rode in the launch
{
    static bool attr_set = false;
    const size_t smem = 2 * (size_t)(DP + 2) * TileCols<T, DP, CS>::value * sizeof(T);
    if (!attr_set) {
        cudaFuncSetAttribute(update_kernel<T, DP, CS, XF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attr_set = true;
    }
    const int nrows = (leg == LEG_F) ? P.n : P.m;
    const int lanes = width < 1 ? 1 : width;
    const bool guard_pool = leg == LEG_V && P.guard > 0.0;       // extra grid rows: the guard band's float64 re-evaluation
    if constexpr (sizeof(T) == 8 && XF == 1 && DP <= 8) {
        // Float64 arguments with few dimensions: four rows per thread halve the shared-memory
        // loads per multiply-add (faster when the grid fills the GPU), two rows give twice the
        // blocks (lower latency when it does not).  Same bits either way, so the choice may follow
        // the width from launch to launch.
        constexpr int RW = 4;
        static bool attr_wide = false;
        if (!attr_wide) {
            cudaFuncSetAttribute(update_kernel<T, DP, CS, XF, RW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            attr_wide = true;
        }
        const int rbw = (UPD_THREADS / 32) * RW * (32 / CS);
        const long long ctas = (long long)((nrows + rbw - 1) / rbw) * lanes;
        if (ctas >= 2 * 148 * 4) {
            const int pool = pool_rows((nrows + rbw - 1) / rbw, guard_pool, lanes);
            launch_pdl(update_kernel<T, DP, CS, XF, RW>, dim3((nrows + rbw - 1) / rbw, lanes + pool), dim3(UPD_THREADS), smem, st, P, leg, lanes);
            return pool > 0;
        }
    }
    if constexpr (sizeof(T) == 4 && DP <= 4 && CS == 4) {
        // Few dimensions, bound by the special-function unit: when a narrow batch would leave SMs
        // without a block, one row per thread gives twice the blocks (same bits, see above).
        static bool attr_narrow = false;
        if (!attr_narrow) {
            cudaFuncSetAttribute(update_kernel<T, DP, CS, XF, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            attr_narrow = true;
        }
        const int rb2 = (UPD_THREADS / 32) * Tune<T, DP>::R * (32 / CS);
        if ((long long)((nrows + rb2 - 1) / rb2) * lanes < NARROW_BLOCKS) {
            const int rbr = (UPD_THREADS / 32) * 1 * (32 / CS);
            const int pool = pool_rows((nrows + rbr - 1) / rbr, guard_pool, lanes);
            launch_pdl(update_kernel<T, DP, CS, XF, 1>, dim3((nrows + rbr - 1) / rbr, lanes + pool), dim3(UPD_THREADS), smem, st, P, leg, lanes);
            return pool > 0;
        }
    }
    const int rb = (UPD_THREADS / 32) * Tune<T, DP>::R * (32 / CS);
    const int pool = pool_rows((nrows + rb - 1) / rb, guard_pool, lanes);
    launch_pdl(update_kernel<T, DP, CS, XF>, dim3((nrows + rb - 1) / rb, lanes + pool), dim3(UPD_THREADS), smem, st, P, leg, lanes);
    return pool > 0;
}

// Several whole cycles per launch: grid.x = row blocks of the larger cloud = one thread-block
// cluster per lane (the caller has checked that a lane has at most MAX_CLUSTER_BLOCKS of them).
template <typename T, int DP, int CS, int XF>
static void launch_cycles(const Dev &P, int cycles, int width, cudaStream_t st)
{
    static bool attr_set = false;
    const size_t smem = 2 * (size_t)(DP + 2) * TileCols<T, DP, CS>::value * sizeof(T);
    if (!attr_set) {
        cudaFuncSetAttribute(lane_cycles_kernel<T, DP, CS, XF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attr_set = true;
    }
    const int rb = (UPD_THREADS / 32) * Tune<T, DP>::R * (32 / CS);
    const int mx = P.n > P.m ? P.n : P.m;
    const int nc = (mx + rb - 1) / rb;
    // a lane small enough to live in shared memory for the whole launch (at four blocks per SM)
    const size_t res_smem = ResidentLayout<T, DP, CS>::bytes(P.n, P.m);
    const bool resident = res_smem <= RESIDENT_SMEM_LIMIT;
    if (resident) {
        static bool res_attr_set = false;
        if (!res_attr_set) {
            cudaFuncSetAttribute(lane_resident_kernel<T, DP, CS, XF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)RESIDENT_SMEM_LIMIT);
            res_attr_set = true;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(nc, width < 1 ? 1 : width); cfg.blockDim = dim3(UPD_THREADS);
    cfg.dynamicSmemBytes = resident ? res_smem : smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = nc; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    if (resident) cudaLaunchKernelEx(&cfg, lane_resident_kernel<T, DP, CS, XF>, P, cycles);
    else cudaLaunchKernelEx(&cfg, lane_cycles_kernel<T, DP, CS, XF>, P, cycles);
}

template <typename T, int DP, int CS>
static bool lane_fits_shared(int n, int m) { return ResidentLayout<T, DP, CS>::bytes(n, m) <= RESIDENT_SMEM_LIMIT; }

#define SKB_V(T, F64, XF, DP, CS) \
    { F64, XF, DP, Tune<T, DP>::R, CS, (UPD_THREADS / 32) * Tune<T, DP>::R * (32 / CS), \
      2 * (size_t)(DP + 2) * TileCols<T, DP, CS>::value * sizeof(T), &launch_update<T, DP, CS, XF>, \
      &launch_cycles<T, DP, CS, XF>, &lane_fits_shared<T, DP, CS> }
#define SKB_ROW(DP) \
    SKB_V(float, 0, 0, DP, 1), SKB_V(float, 0, 0, DP, 4), SKB_V(float, 0, 0, DP, 32), \
    SKB_V(double, 1, 0, DP, 1), SKB_V(double, 1, 0, DP, 4), SKB_V(double, 1, 0, DP, 32), \
    SKB_V(double, 1, 1, DP, 1), SKB_V(double, 1, 1, DP, 4), SKB_V(double, 1, 1, DP, 32)

static const Variant g_variants[] = {SKB_ROW(2), SKB_ROW(3), SKB_ROW(4), SKB_ROW(8), SKB_ROW(16), SKB_ROW(32)};

template <typename T, int XF>
static int launch_bigd(const Dev &P, int leg, int width, cudaStream_t st)
{
    static bool attr_set = false;
    const size_t smem = 2 * (size_t)BIGD_KC * (BIGD_RB + BIGD_TJ) * sizeof(T);
    if (!attr_set) {
        cudaFuncSetAttribute(update_bigd_kernel<T, XF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attr_set = true;
    }
    const int nrows = (leg == LEG_F) ? P.n : P.m;
    dim3 grid((nrows + BIGD_RB - 1) / BIGD_RB, width < 1 ? 1 : width);
    launch_pdl(update_bigd_kernel<T, XF>, grid, dim3(UPD_THREADS), smem, st, P, leg);
    return 0;                       // no pool in this kernel
}

// DP = 0 marks the large-d kernels: the padded dimension is d rounded up to the chunk size
static const Variant g_bigd[] = {
    {0, 0, 0, 4, 4, BIGD_RB, 2 * (size_t)BIGD_KC * (BIGD_RB + BIGD_TJ) * 4, &launch_bigd<float, 0>, nullptr, nullptr},
    {1, 0, 0, 4, 4, BIGD_RB, 2 * (size_t)BIGD_KC * (BIGD_RB + BIGD_TJ) * 8, &launch_bigd<double, 0>, nullptr, nullptr},
    {1, 1, 0, 4, 4, BIGD_RB, 2 * (size_t)BIGD_KC * (BIGD_RB + BIGD_TJ) * 8, &launch_bigd<double, 1>, nullptr, nullptr},
};

int padded_dim(int d)
{
    if (d > 32) return d <= 1024 ? (d + BIGD_KC - 1) / BIGD_KC * BIGD_KC : -1;
    const int opts[] = {2, 3, 4, 8, 16, 32};
    for (int o : opts) if (d <= o) return o;
    return -1;
}

const Variant *choose_variant(int W, int n, int m, int d, bool f64, bool fast_exp, int force_cs)
{
    const int DP = padded_dim(d);
    if (DP < 0) return nullptr;
    if (d > 32) {
        for (const Variant &v : g_bigd)
            if (v.f64 == (f64 ? 1 : 0) && v.xf == ((f64 && fast_exp) ? 1 : 0)) return &v;
        return nullptr;
    }
    const int mn = n < m ? n : m;
    int R = 2;
    for (const Variant &v : g_variants)
        if (v.f64 == (f64 ? 1 : 0) && v.DP == DP) { R = v.R; break; }
    // smallest column split that fills its CTAs' rows and gives every SM about four CTAs
    int cs = 32;
    double best = -1.0;
    for (int c : {1, 4, 32}) {
        const int rb = (UPD_THREADS / 32) * R * (32 / c);
        long long ctas = (long long)W * ((mn + rb - 1) / rb);
        if (!f64 && DP <= 4 && c == 4) {             // the launcher may drop to one row per thread
            const int rb1 = (UPD_THREADS / 32) * (32 / c);
            ctas = (long long)W * ((mn + rb1 - 1) / rb1);
        }
        const double util_n = (double)n / ((double)((n + rb - 1) / rb) * rb);
        const double util_m = (double)m / ((double)((m + rb - 1) / rb) * rb);
        const double fill = ctas >= 592 ? 1.0 : (double)ctas / 592.0;
        // a whole lane per CTA (c == 1) is marginally faster at full width but leaves the narrow tail of
        // an active batch to one CTA per lane, so it only wins when the 4-way split would idle rows
        const double score = (util_n < util_m ? util_n : util_m) * fill * (c == 32 ? 0.6 : (c == 1 ? 0.85 : 1.0));
        if (score > best + 1e-9) { best = score; cs = c; }
    }
    if (force_cs == 1 || force_cs == 4 || force_cs == 32) cs = force_cs;
    for (const Variant &v : g_variants)
        if (v.f64 == (f64 ? 1 : 0) && v.xf == ((f64 && fast_exp) ? 1 : 0) && v.DP == DP && v.CS == cs) return &v;
    return nullptr;
}

// The guard band's float64 re-evaluation as a launch of its own (deep lanes, whose update kernels carry
// no pool): about two blocks per SM look for lanes whose fused screen lies in the band and share each
// one's rows.  It sits between the column check and the planner in the chain and, like every kernel of
// the chain, waits for its predecessor before it reads anything.
__global__ void __launch_bounds__(UPD_THREADS) guard_pool_kernel(const Dev P)
{
    __shared__ unsigned long long red[UPD_THREADS / 32];
    pdl_enter();
    const Ctl c = *P.ctl;
    guard_pool<true>(P, c, 0, red);        // with the 16-byte loads for deep bf16 lanes
}

void launch_guard_pool(const Dev &P, cudaStream_t st)
{
    launch_pdl(guard_pool_kernel, dim3(2 * 148, 1), dim3(UPD_THREADS), 0, st, P);
}

}  // namespace skb
