// Host side of the C ABI: validation, workspace carving, the cycle enqueue loop and the
// asynchronous width read-back.  No device memory is allocated here; the only CUDA
// objects a handle holds are two events and a small pinned host block borrowed from a pool
// (plus its own timing events once phase timing has been switched on).
#include <nvtx3/nvToolsExt.h>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/sinkhorn_batch.h"
#include "skb_host.h"

using namespace skb;

struct skb_batch {
    Dev dev;
    skb_config cfg;
    const Variant *var;
    cudaStream_t stream;
    Ctl *h_ctl;            // pinned, 2 snapshots
    cudaEvent_t ev[2];
    int known_width;       // last physical width the host has seen
    bool finished;
    long long enqueued;    // cycles enqueued so far
    long long launches;    // kernels launched so far
    int res_device;        // device the pooled host resources belong to
    bool tensor;           // the tensor-core update kernel is in use
    bool snap_pending;     // step() left a control-block snapshot in flight (ev[snap_idx])
    int snap_idx;
    // phase timing (Eq. 11's cost record): off unless sinkhorn_batch_set_profiling turned it on
    bool profiling;
    int lanes_used;        // lanes the batch has taken in so far (create: W; each refill adds to it)
    long long enqueued_at_refill;   // cycles enqueued when the last lanes came in (the drain cap counts from there)
    bool no_multi_cycle;   // measurement switch: keep one launch per leg even where several cycles per launch are possible
    std::vector<cudaEvent_t> pev;      // timing events, PHASE_EVENTS_PER_CYCLE per enqueued cycle of a chunk + 1
    int pev_used;                      // events recorded since the last harvest
    float phase_ms[SKB_N_PHASES];
    std::vector<float> cycle_update_ms;   // per cycle: f-leg + g-leg
    alignas(64) unsigned char maps[2 * 128];   // CUtensorMap of x and of y
    GuardList guards;      // guard strips of the workspace in the layout the batch runs in
    std::string err;
};

static skb_status poll_snapshot(skb_batch *h, bool wait);
static skb_status read_ctl(skb_batch *h, Ctl *c);

// Text of the last failed create (or host-buffer solve) of the calling thread.
static thread_local std::string g_create_err;

// NVTX ranges around the host-side phases (create, step, drain and its chunks, refill): they cost a
// few nanoseconds when no tool is attached and give a timeline tool the structure of a solve.
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange &) = delete;
    NvtxRange &operator=(const NvtxRange &) = delete;
};
static const int PHASE_EVENTS_PER_CYCLE = 5;     // f-leg | column check | plan | emit/move | g-leg, boundaries shared
static const int PROFILE_CHUNK = 16;             // cycles between two harvests of the timing events

// Host-side resources of a handle (a pinned control-block pair and two events) are recycled
// through a small per-device pool: allocating and freeing pinned memory costs hundreds of
// microseconds, which would dominate short solves created in a loop.
struct HostRes { Ctl *pinned; cudaEvent_t ev[2]; int device; };
static std::mutex g_pool_mu;
static std::vector<HostRes> g_pool;

static cudaError_t host_res_get(HostRes *r)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    {
        std::lock_guard<std::mutex> lk(g_pool_mu);
        for (size_t i = 0; i < g_pool.size(); ++i)
            if (g_pool[i].device == dev) { *r = g_pool[i]; g_pool.erase(g_pool.begin() + i); return cudaSuccess; }
    }
    r->device = dev; r->pinned = nullptr; r->ev[0] = r->ev[1] = nullptr;
    if ((e = cudaHostAlloc((void **)&r->pinned, 2 * sizeof(Ctl), cudaHostAllocDefault)) != cudaSuccess) return e;
    if ((e = cudaEventCreate(&r->ev[0])) != cudaSuccess) return e;      // timing events: they also bracket create
    return cudaEventCreate(&r->ev[1]);
}

static void host_res_put(const HostRes &r)
{
    std::lock_guard<std::mutex> lk(g_pool_mu);
    if (g_pool.size() < 64) { g_pool.push_back(r); return; }
    if (r.ev[0]) cudaEventDestroy(r.ev[0]);
    if (r.ev[1]) cudaEventDestroy(r.ev[1]);
    if (r.pinned) cudaFreeHost(r.pinned);
}

// fp32 arithmetic: the expanded cost |x|^2+|y|^2-2x.y carries an error of about one ulp of the
// scaled squared radius M = s*max|x-c|^2 into every exponent.  Above FORM_DIFF_RADIUS a lane
// switches to the difference form; above mixed_radius(tol) (any lane) an automatic batch computes
// its exponents in float64 and only the exponentials in fp32.
static const double FORM_DIFF_RADIUS = 512.0;
static const double MIXED_RADIUS = 512.0;
// One ulp of M in the exponent is a relative error of about M * 8e-8 in every plan entry and, where it
// is systematic, in the residuals: 4 % of a tolerance of 1e-3 at M = 512.  A stricter tolerance lowers
// the radius in proportion, so that the evaluation error stays the same fraction of the threshold.
static double mixed_radius(double tol)
{
    return MIXED_RADIUS * (tol < 1.0e-3 ? tol / 1.0e-3 : 1.0);
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static bool config_ok(const skb_config *c, std::string &why)
{
    if (!c) { why = "config is null"; return false; }
    if (c->W < 1 || c->n < 1 || c->m < 1 || c->d < 1) { why = "W, n, m, d must be >= 1"; return false; }
    if (c->xy_dtype != SKB_F32 && c->xy_dtype != SKB_BF16) { why = "bad xy_dtype"; return false; }
    if (c->mode < SKB_ACTIVE || c->mode > SKB_MASKED_EXIT) { why = "bad mode"; return false; }
    if (c->compute < SKB_COMPUTE_AUTO || c->compute > SKB_COMPUTE_TENSOR) { why = "bad compute type"; return false; }
    if (c->max_iter < 1 || c->audit_every < 1) { why = "max_iter and audit_every must be >= 1"; return false; }
    if (c->cost_form < 0 || c->cost_form > 2) { why = "cost_form must be 0 (automatic), 1 (expanded) or 2 (difference)"; return false; }
    if (c->column_split != 0 && c->column_split != 1 && c->column_split != 4 && c->column_split != 32) {
        why = "column_split must be 0, 1, 4 or 32"; return false;
    }
    if (c->lane_capacity != 0 && c->lane_capacity < c->W) { why = "lane_capacity must be 0 (= W) or at least W"; return false; }
    if (c->lane_capacity > c->W && c->mode != SKB_ACTIVE) { why = "finished lanes can only be replaced in ACTIVE mode"; return false; }
    if (!(c->guard_band <= 0.5f)) { why = "guard_band must be at most 0.5 (negative: off, 0: default)"; return false; }
    return true;
}

// Relative half-width of the guard band: the configured value, off when negative; when left at 0 it is
// 2.5e-4 for d <= 32 and off for deeper lanes, where the float64 re-evaluation of one lane is half a
// GFLOP (d = 512, n = m = 1024) and the tensor path's own evaluation error would need a band of a
// per cent: there the caller names the width it is willing to pay for.
static double guard_width(const skb_config *c)
{
    if (c->guard_band < 0.0f) return 0.0;
    if (c->guard_band > 0.0f) return (double)c->guard_band;
    return c->d > 32 ? 0.0 : 2.5e-4;
}

// Lays the batch's arrays out in the workspace (base may be null: size query only).
// Every array is followed by a guard strip (GUARD_STRIP_BYTES of a known pattern, see
// sinkhorn_batch_check_guards); their offsets are listed in *guards.
static size_t carve(const skb_config *c, const Variant *var, bool tensor, char *base, Dev *D, size_t *zero_end_out = nullptr,
                    GuardList *guards = nullptr)
{
    size_t off = 0;
    int strips = 0;
    auto take = [&](size_t bytes) -> void * {
        void *p = base ? base + off : nullptr;
        off += align_up(bytes, 256);
        if (guards && strips < MAX_GUARD_STRIPS) guards->off256[strips] = (unsigned)(off / 256);
        ++strips;
        off += GUARD_STRIP_BYTES;
        return p;
    };
    const size_t W = c->W, n = c->n, m = c->m;
    const size_t L = c->lane_capacity > c->W ? c->lane_capacity : c->W;      // lanes the result buffers hold
    const size_t np = align_up(n, 4), mp = align_up(m, 4), DP = var->DP ? var->DP : padded_dim(c->d);
    const size_t ts = var->f64 ? 8 : 4;
    Dev d;
    memset(&d, 0, sizeof(d));
    d.L = (int)L;
    d.W = c->W; d.n = c->n; d.m = c->m; d.d = c->d; d.np = (int)np; d.mp = (int)mp; d.DP = (int)DP;
    d.mode = c->mode == SKB_MASKED_EXIT ? (int)MODE_MASKED : (int)c->mode;
    d.early_exit = c->mode == SKB_MASKED_EXIT;
    d.max_iter = c->max_iter; d.audit_every = c->audit_every;
    d.xy_bf16 = c->xy_dtype == SKB_BF16; d.compute_f64 = var->f64;
    d.cost_form = c->d > 32 ? 1 : c->cost_form;      // the large-d kernels only have the expanded form
    // fp32: above this scaled squared radius the expanded cost loses more than ~4e-6 per term
    d.form_threshold = FORM_DIFF_RADIUS;
    // control block first, then everything that must start at zero, in one contiguous range
    d.ctl = (Ctl *)take(sizeof(Ctl));
    d.guard_bad = (int *)take(4);
    d.state = (int *)take(W * 4); d.flag = (int *)take(W * 4); d.verdict = (int *)take(W * 4);
    d.nonfinite = (int *)take(W * 4);
    d.ret_at = (int *)take(W * 4); d.n_checks = (int *)take(W * 4);
    d.rsum_row64 = (unsigned long long *)take(W * 8); d.esc = (int *)take(W * 4);
    d.rsum_row = (unsigned long long *)take(W * 8); d.rsum_col = (unsigned long long *)take(W * 8);
    d.depth = (int *)take(L * 4); d.status = (int *)take(L * 4); d.emitted = (int *)take(L * 4);
    d.res_row = (double *)take(L * 8); d.res_col = (double *)take(L * 8);
    d.start = (int *)take(W * 4);
    d.rrow = (double *)take(W * 8); d.rcol = (double *)take(W * 8);
    // widths[k] of every cycle the batch can run: max_iter per generation of lanes
    d.widths_cap = (int)(((size_t)c->max_iter + 1) * ((L + W - 1) / W) + 1);
    d.widths = (int *)take((size_t)d.widths_cap * 4);
    const size_t nblk128 = ((n > m ? n : m) + 127) / 128;
    d.tc_cnt = (unsigned *)take(W * nblk128 * 4);     // in every layout, so that the zeroed range is the same for all
    const size_t zero_end = off;
    d.scale = (double *)take(W * 8); d.lane_id = (int *)take(W * 4);
    d.center = (double *)take(W * DP * 8); d.form = (int *)take(W * 4);
    d.ret_slot = (int *)take(W * 4); d.ret_lane = (int *)take(W * 4); d.ret_src = (int *)take(W * 4);
    d.ret_scale = (double *)take(W * 8);
    d.hole_list = (int *)take(W * 4); d.fill_list = (int *)take(W * 4);
    d.tensor = tensor ? 1 : 0;
    if (tensor) {
        d.xb = take(tc_tiled_bytes(c->W, c->n, c->d)); d.yb = take(tc_tiled_bytes(c->W, c->m, c->d));
        d.tc_pm = (float *)take(W * nblk128 * 2 * TC_MAX_SPLIT * 128 * 4);
        d.tc_ps = (double *)take(W * nblk128 * 2 * TC_MAX_SPLIT * 128 * 8);
    } else {
        d.xs = take(W * DP * np * ts); d.ys = take(W * DP * mp * ts);
    }
    d.ft[0] = take(W * np * ts); d.ft[1] = take(W * np * ts); d.gt = take(W * mp * ts);
    d.fl[0] = take(W * np * ts); d.fl[1] = take(W * np * ts); d.gl = take(W * mp * ts);
    d.sqx = (double *)take(W * np * 8); d.sqy = (double *)take(W * mp * 8);
    d.la2 = (double *)take(W * np * 8); d.lb2 = (double *)take(W * mp * 8);
    d.wa = (double *)take(W * np * 8); d.wb = (double *)take(W * mp * 8);
    d.phi[0] = (double *)take(W * np * 8); d.phi[1] = (double *)take(W * np * 8);
    d.gam = (double *)take(W * mp * 8);
    d.f_out = (double *)take(L * n * 8); d.g_out = (double *)take(L * m * 8);
    // guard band: raw copies of the inputs (the float64 re-evaluation reads nothing but these and the potentials)
    d.guard = guard_width(c);
    if (d.guard > 0.0) {
        const size_t es = c->xy_dtype == SKB_BF16 ? 2 : 4;
        d.xraw_stride = align_up(n * (size_t)c->d * es, 16); d.yraw_stride = align_up(m * (size_t)c->d * es, 16);
        d.xraw = take(W * d.xraw_stride); d.yraw = take(W * d.yraw_stride);
    }
    if (D) { *D = d; D->tol_screen = 0; D->tol_stop = 0; }
    if (zero_end_out) *zero_end_out = zero_end;
    if (guards) guards->count = strips <= MAX_GUARD_STRIPS ? strips : 0;      // more arrays than the list holds: no strips checked
    return off;
}

static const Variant *variant_for(const skb_config *c, int compute)
{
    if (compute == SKB_COMPUTE_TENSOR) compute = SKB_COMPUTE_F32;     // fp32 epilogue, same scratch shapes
    const bool f64 = compute == SKB_COMPUTE_F64 || compute == SKB_COMPUTE_MIXED;
    return choose_variant(c->W, c->n, c->m, c->d, f64, compute == SKB_COMPUTE_MIXED, c->column_split);
}

extern "C" size_t sinkhorn_batch_workspace_bytes(const skb_config *cfg)
{
    std::string why;
    if (!config_ok(cfg, why)) return 0;
    // an automatic batch may end up with float64 coordinates: size for the larger layout
    if (cfg->compute == SKB_COMPUTE_TENSOR && !tc_eligible(cfg->d, cfg->xy_dtype == SKB_BF16)) return 0;
    const Variant *v = variant_for(cfg, cfg->compute == SKB_COMPUTE_AUTO ? SKB_COMPUTE_MIXED : cfg->compute);
    if (!v) return 0;
    size_t need = carve(cfg, v, cfg->compute == SKB_COMPUTE_TENSOR, nullptr, nullptr);
    if (cfg->compute == SKB_COMPUTE_AUTO && tc_eligible(cfg->d, cfg->xy_dtype == SKB_BF16)) {
        const size_t t = carve(cfg, variant_for(cfg, SKB_COMPUTE_F32), true, nullptr, nullptr);
        if (t > need) need = t;
    }
    return need;
}

static skb_status fail(skb_batch *h, skb_status st, const std::string &msg)
{
    if (h) h->err = msg; else g_create_err = msg;
    return st;
}

static skb_status cuda_fail(skb_batch *h, cudaError_t e, const char *where)
{
    return fail(h, SKB_ERR_CUDA, std::string(where) + ": " + cudaGetErrorString(e));
}

extern "C" skb_status sinkhorn_batch_create(const void *x, const void *y, const float *a, const float *b,
                                            const float *eps, float tol, const skb_config *cfg, skb_batch **out)
{
    NvtxRange nvtx_range("skb:create");
    if (!out) return fail(nullptr, SKB_ERR_NULL, "out is null");
    *out = nullptr;
    if (!x || !y || !a || !b || !eps || !cfg) return fail(nullptr, SKB_ERR_NULL, "x, y, a, b, eps and cfg are required");
    std::string why;
    if (!config_ok(cfg, why)) {
        const bool shape = cfg->W < 1 || cfg->n < 1 || cfg->m < 1 || cfg->d < 1;
        return fail(nullptr, shape ? SKB_ERR_SHAPE : SKB_ERR_VALUE, why);
    }
    if (!(tol > 0.0f) || !std::isfinite(tol)) return fail(nullptr, SKB_ERR_VALUE, "tol must be positive and finite");
    const bool automatic = cfg->compute == SKB_COMPUTE_AUTO;
    const Variant *var = variant_for(cfg, automatic ? SKB_COMPUTE_F32 : cfg->compute);
    const Variant *var_big = variant_for(cfg, automatic ? SKB_COMPUTE_MIXED : cfg->compute);
    if (!var || !var_big) return fail(nullptr, SKB_ERR_SHAPE, "dimension d is not supported by any update kernel");
    const int mx = cfg->n > cfg->m ? cfg->n : cfg->m;
    // a lane's residual is a 64-bit fixed-point sum of per-row terms clamped at RSUM_ROW_MAX
    if ((double)mx * RSUM_ROW_MAX * RSUM_SCALE >= 18446744073709551616.0)
        return fail(nullptr, SKB_ERR_SHAPE, "n and m must be at most 262143 (fixed-point residual sums)");
    if (cfg->W > 65535) return fail(nullptr, SKB_ERR_SHAPE, "W must be <= 65535");
    const bool can_tensor = tc_eligible(cfg->d, cfg->xy_dtype == SKB_BF16);
    if (cfg->compute == SKB_COMPUTE_TENSOR && !can_tensor)
        return fail(nullptr, SKB_ERR_SHAPE, "the tensor-core path needs bf16 x, y and d a multiple of 64 with 64 <= d <= 512");
    size_t zero_end = 0;
    carve(cfg, var_big, false, nullptr, nullptr, &zero_end);
    const size_t need = sinkhorn_batch_workspace_bytes(cfg);
    if (!cfg->workspace) return fail(nullptr, SKB_ERR_WORKSPACE, "workspace is null");
    if (((uintptr_t)cfg->workspace & 255u) != 0) return fail(nullptr, SKB_ERR_WORKSPACE, "workspace must be 256-byte aligned");
    if (cfg->workspace_bytes < need) {
        char buf[128];
        snprintf(buf, sizeof(buf), "workspace too small: %zu bytes given, %zu needed", cfg->workspace_bytes, need);
        return fail(nullptr, SKB_ERR_WORKSPACE, buf);
    }
    skb_batch *h = new (std::nothrow) skb_batch();
    if (!h) return fail(nullptr, SKB_ERR_CUDA, "host allocation failed");
    h->cfg = *cfg; h->var = var; h->stream = (cudaStream_t)cfg->stream;
    h->known_width = cfg->W; h->finished = false; h->enqueued = 0; h->launches = 0; h->h_ctl = nullptr;
    h->ev[0] = h->ev[1] = nullptr;
    h->tensor = cfg->compute == SKB_COMPUTE_TENSOR;
    h->snap_pending = false; h->snap_idx = 0; h->profiling = false; h->pev_used = 0; h->no_multi_cycle = false;
    h->lanes_used = cfg->W; h->enqueued_at_refill = 0;
    for (int i = 0; i < SKB_N_PHASES; ++i) h->phase_ms[i] = 0.f;
    h->guards.count = 0;
    carve(cfg, var, h->tensor, (char *)cfg->workspace, &h->dev, nullptr, &h->guards);
    h->dev.tol_stop = (double)tol;
    h->dev.tol_screen = cfg->tol_screen > 0.0f ? (double)cfg->tol_screen : (double)tol;
    cudaError_t e;
    HostRes res;
    e = host_res_get(&res);
    h->h_ctl = res.pinned; h->ev[0] = res.ev[0]; h->ev[1] = res.ev[1]; h->res_device = res.device;
    if (e != cudaSuccess) {
        skb_status st = cuda_fail(nullptr, e, "create");
        sinkhorn_batch_destroy(h);
        return st;
    }
    memset(h->h_ctl, 0, 2 * sizeof(Ctl));
    Ctl init;
    memset(&init, 0, sizeof(init));
    init.n_phys = cfg->W; init.n_running = cfg->W;
    h->h_ctl[0] = init;
    cudaEventRecord(h->ev[1], h->stream);          // start of the set-up work (SKB_PHASE_CREATE)
    if ((e = cudaMemsetAsync(cfg->workspace, 0, zero_end, h->stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(h->dev.ctl, &h->h_ctl[0], sizeof(Ctl), cudaMemcpyHostToDevice, h->stream)) != cudaSuccess) {
        skb_status st = cuda_fail(nullptr, e, "create");
        sinkhorn_batch_destroy(h);
        return st;
    }
    launch_lane_stats(h->dev, x, y, eps, 0, 0, cfg->W, 0, h->stream);
    h->launches += 2;   // lane statistics + layout kernel
    if (automatic) {
        // read the largest scaled radius back and pick the arithmetic for the whole batch
        if ((e = cudaMemcpyAsync(&h->h_ctl[1], h->dev.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost, h->stream)) != cudaSuccess ||
            (e = cudaStreamSynchronize(h->stream)) != cudaSuccess) {
            skb_status st = cuda_fail(nullptr, e, "create");
            sinkhorn_batch_destroy(h);
            return st;
        }
        double radius;
        memcpy(&radius, &h->h_ctl[1].max_radius_bits, sizeof(double));
        const double ts = h->dev.tol_stop, tsc = h->dev.tol_screen;
        if (radius > mixed_radius(ts < tsc ? ts : tsc)) {
            h->var = var_big;
            carve(cfg, var_big, false, (char *)cfg->workspace, &h->dev, nullptr, &h->guards);
        } else if (can_tensor) {
            h->tensor = true;
            carve(cfg, var, true, (char *)cfg->workspace, &h->dev, nullptr, &h->guards);
        }
        h->dev.tol_stop = ts; h->dev.tol_screen = tsc;
    }
    launch_guard_strips(cfg->workspace, h->guards, true, nullptr, h->stream);      // the layout is final from here on
    h->launches += 1;
    if (h->tensor) {
        // the MMA operands: tiled copies of x and y that the compaction may permute
        const char *why = nullptr;
        launch_retile(x, h->dev.xb, cfg->W, cfg->n, cfg->d, h->stream);
        launch_retile(y, h->dev.yb, cfg->W, cfg->m, cfg->d, h->stream);
        h->launches += 2;
        if ((why = tc_make_map(h->maps, h->dev.xb, cfg->W, cfg->n, cfg->d)) != nullptr ||
            (why = tc_make_map(h->maps + 128, h->dev.yb, cfg->W, cfg->m, cfg->d)) != nullptr) {
            skb_status st = fail(nullptr, SKB_ERR_CUDA, why);
            sinkhorn_batch_destroy(h);
            return st;
        }
    }
    launch_prep(h->dev, x, y, a, b, 0, cfg->W, h->stream);
    if (h->dev.guard > 0.0) {
        const size_t es = cfg->xy_dtype == SKB_BF16 ? 2 : 4;
        const size_t xb = (size_t)cfg->n * cfg->d * es, yb = (size_t)cfg->m * cfg->d * es;
        if ((e = cudaMemcpy2DAsync(h->dev.xraw, h->dev.xraw_stride, x, xb, xb, cfg->W, cudaMemcpyDeviceToDevice, h->stream)) != cudaSuccess ||
            (e = cudaMemcpy2DAsync(h->dev.yraw, h->dev.yraw_stride, y, yb, yb, cfg->W, cudaMemcpyDeviceToDevice, h->stream)) != cudaSuccess) {
            skb_status st = cuda_fail(nullptr, e, "create (raw input copies)");
            sinkhorn_batch_destroy(h);
            return st;
        }
    }
    // the pinned block is reused for snapshots: wait until the initial copy has been consumed
    if ((e = cudaEventRecord(h->ev[0], h->stream)) != cudaSuccess || (e = cudaGetLastError()) != cudaSuccess) {
        skb_status st = cuda_fail(nullptr, e, "create");
        sinkhorn_batch_destroy(h);
        return st;
    }
    if ((e = cudaEventSynchronize(h->ev[0])) != cudaSuccess ||
        (e = cudaEventElapsedTime(&h->phase_ms[SKB_PHASE_CREATE], h->ev[1], h->ev[0])) != cudaSuccess) {
        skb_status st = cuda_fail(nullptr, e, "create");
        sinkhorn_batch_destroy(h);
        return st;
    }
    *out = h;
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_warm_start(skb_batch *h, const double *f0, const double *g0, int audit_initial)
{
    if (!h) return SKB_ERR_NULL;
    if (h->enqueued != 0) return fail(h, SKB_ERR_STATE, "a warm proposal must be given before the first step or drain");
    if (f0 || g0) { launch_warm(h->dev, f0, g0, h->stream); h->launches += 1; }
    h->dev.audit_initial = audit_initial ? 1 : 0;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : cuda_fail(h, e, "warm_start");
}

extern "C" skb_status sinkhorn_batch_refill(skb_batch *h, const void *x, const void *y, const float *a, const float *b,
                                            const float *eps, int count, int *first_lane)
{
    NvtxRange nvtx_range("skb:refill");
    if (!h) return SKB_ERR_NULL;
    if (!x || !y || !a || !b || !eps) return fail(h, SKB_ERR_NULL, "x, y, a, b and eps are required");
    if (count < 1) return fail(h, SKB_ERR_VALUE, "count must be >= 1");
    if (h->cfg.mode != SKB_ACTIVE) return fail(h, SKB_ERR_STATE, "finished lanes can only be replaced in ACTIVE mode");
    if (h->lanes_used + count > h->dev.L) {
        char buf[128];
        snprintf(buf, sizeof(buf), "lane capacity exhausted: %d lanes taken in, %d more asked, capacity %d", h->lanes_used, count, h->dev.L);
        return fail(h, SKB_ERR_SHAPE, buf);
    }
    skb_status st0 = poll_snapshot(h, true);
    if (st0 != SKB_OK) return st0;
    Ctl c;
    st0 = read_ctl(h, &c);                           // synchronises: the free slots are those past the device's width
    if (st0 != SKB_OK) return st0;
    const int width = c.n_phys;                      // 0 once everything has finished (ACTIVE: the width is the survivors)
    if (width + count > h->cfg.W) {
        char buf[128];
        snprintf(buf, sizeof(buf), "%d slots are free, %d lanes offered", h->cfg.W - width, count);
        return fail(h, SKB_ERR_STATE, buf);
    }
    const Dev &D = h->dev;
    const size_t es = h->cfg.xy_dtype == SKB_BF16 ? 2 : 4;
    launch_lane_stats(D, x, y, eps, width, h->lanes_used, count, c.cycle, h->stream);
    cudaError_t e = cudaSuccess;
    if (h->tensor) {
        const size_t xt = tc_tiled_bytes(1, h->cfg.n, h->cfg.d), yt = tc_tiled_bytes(1, h->cfg.m, h->cfg.d);
        launch_retile(x, (char *)D.xb + (size_t)width * xt, count, h->cfg.n, h->cfg.d, h->stream);
        launch_retile(y, (char *)D.yb + (size_t)width * yt, count, h->cfg.m, h->cfg.d, h->stream);
        h->launches += 2;
    }
    launch_prep(D, x, y, a, b, width, count, h->stream);
    if (D.guard > 0.0) {
        const size_t xb = (size_t)h->cfg.n * h->cfg.d * es, yb = (size_t)h->cfg.m * h->cfg.d * es;
        e = cudaMemcpy2DAsync((char *)D.xraw + (size_t)width * D.xraw_stride, D.xraw_stride, x, xb, xb, count, cudaMemcpyDeviceToDevice, h->stream);
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync((char *)D.yraw + (size_t)width * D.yraw_stride, D.yraw_stride, y, yb, yb, count, cudaMemcpyDeviceToDevice, h->stream);
    }
    launch_refill_ctl(D, count, h->stream);
    h->launches += 3;
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e, "refill");
    if (first_lane) *first_lane = h->lanes_used;
    h->lanes_used += count;
    h->known_width = width + count;
    h->finished = false;
    h->enqueued_at_refill = h->enqueued;
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_set_profiling(skb_batch *h, int on)
{
    if (!h) return SKB_ERR_NULL;
    if (h->enqueued != 0) return fail(h, SKB_ERR_STATE, "phase timing must be switched before the first step or drain");
    if (on && h->pev.empty()) {
        h->pev.resize(PROFILE_CHUNK * PHASE_EVENTS_PER_CYCLE + 1, nullptr);
        for (cudaEvent_t &ev : h->pev) {
            cudaError_t e = cudaEventCreate(&ev);
            if (e != cudaSuccess) return cuda_fail(h, e, "set_profiling");
        }
    }
    h->profiling = on != 0;
    return SKB_OK;
}

// one full cycle: f-leg (+ row screen of the previous state), column check of screen-positive
// lanes, plan, emit/compact, g-leg
// Returns 1 if a column-check launch carried the guard band's pool.
static int launch_leg(skb_batch *h, int leg, int w)
{
    if (h->tensor) { launch_update_tc(h->dev, h->maps, leg, w, h->stream); return 0; }
    return h->var->launch(h->dev, leg, w, h->stream);
}

// ACTIVE batches whose lanes have few row blocks run several whole cycles per launch, one
// thread-block cluster per lane (lane_cycles_kernel), followed by one planner for all of them.
static bool cycles_in_one_launch(const skb_batch *h)
{
    if (h->cfg.mode != SKB_ACTIVE || h->tensor || h->profiling || !h->var->launch_cycles || h->no_multi_cycle) return false;
    const int mx = h->cfg.n > h->cfg.m ? h->cfg.n : h->cfg.m;
    const int nc = (mx + h->var->rows_per_cta - 1) / h->var->rows_per_cta;
    if (nc > MAX_CLUSTER_BLOCKS) return false;
    // Lanes too large for shared memory run the streaming version, which is worth it once the batch is
    // down to about one wave of blocks (it saves launches, not traffic); a wide batch of such lanes is
    // better served by one launch per leg (sensor at 256 lanes: 1.12 against 1.20 ms per solve).
    if (!h->var->lane_fits_shared(h->cfg.n, h->cfg.m) && (long long)h->known_width * nc > 148 * 4) return false;
    return true;
}

// `cycles` cycles in one launch (1 <= cycles <= MAX_CYCLES_IN_LAUNCH): lanes that pass inside it write their own
// outputs; the planner accounts for every cycle of the launch and fills the holes.
static void enqueue_cycles_launch(skb_batch *h, int cycles)
{
    const int w = h->known_width;
    h->var->launch_cycles(h->dev, cycles, w, h->stream);
    int nk = 1;
    nk += launch_plan_cycles(h->dev, w, cycles, h->stream);
    nk += launch_emit_move(h->dev, w, h->stream);
    h->enqueued += cycles;
    h->launches += nk;
}

static void enqueue_cycle(skb_batch *h)
{
    if (cycles_in_one_launch(h)) { enqueue_cycles_launch(h, 1); return; }
    const int w = h->known_width;
    // phase timing: an event between every two kernels of the cycle (which also keeps them from
    // overlapping: a kernel launched after an event record waits for everything before it)
    const bool prof = h->profiling && h->pev_used + PHASE_EVENTS_PER_CYCLE + (h->pev_used == 0 ? 1 : 0) <= (int)h->pev.size();
    auto mark = [&]() { if (prof) cudaEventRecord(h->pev[h->pev_used++], h->stream); };
    if (prof && h->pev_used == 0) mark();
    launch_leg(h, LEG_F, w); mark();
    const int pool_rode = launch_leg(h, LEG_V, w);
    int nk = 3;
    if (h->dev.guard > 0.0 && !pool_rode) {
        // deep lanes (their update kernels carry no pool) and batches so wide that the column check's
        // grid has no rows to spare: the guard band's re-evaluation is a launch of its own
        launch_guard_pool(h->dev, h->stream);
        ++nk;
    }
    mark();
    nk += launch_plan(h->dev, w, h->stream); mark();
    nk += launch_emit_move(h->dev, w, h->stream); mark();
    launch_leg(h, LEG_G, w); mark();
    h->enqueued++;
    h->launches += nk;
}

// Waits for the timing events recorded so far and adds their intervals to the phase totals.
static cudaError_t harvest_phases(skb_batch *h)
{
    if (h->pev_used < 2) { h->pev_used = 0; return cudaSuccess; }
    cudaError_t e = cudaEventSynchronize(h->pev[h->pev_used - 1]);
    static const int phase_of[PHASE_EVENTS_PER_CYCLE] = {SKB_PHASE_F_LEG, SKB_PHASE_COLUMN_CHECK, SKB_PHASE_PLAN,
                                                         SKB_PHASE_EMIT_MOVE, SKB_PHASE_G_LEG};
    float upd = 0.f;
    for (int i = 0; i + 1 < h->pev_used && e == cudaSuccess; ++i) {
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, h->pev[i], h->pev[i + 1]);
        const int ph = phase_of[i % PHASE_EVENTS_PER_CYCLE];
        h->phase_ms[ph] += ms;
        if (ph == SKB_PHASE_F_LEG || ph == SKB_PHASE_G_LEG) upd += ms;
        if (ph == SKB_PHASE_G_LEG) { h->cycle_update_ms.push_back(upd); upd = 0.f; }
    }
    h->pev_used = 0;
    return e;
}

static skb_status absorb(skb_batch *h, const Ctl &c)
{
    if (c.error & ERR_VALUE) return fail(h, SKB_ERR_VALUE, "inputs rejected on the device: weights and eps must be positive, coordinates finite");
    if (c.error & ERR_WAIT) return fail(h, SKB_ERR_CUDA, "a bounded wait inside a kernel ran out (pipeline barrier never completed)");
    if (c.error) return fail(h, SKB_ERR_CUDA, "a kernel reported an internal error");
    if (h->cfg.mode == SKB_ACTIVE && c.n_phys >= 0 && c.n_phys < h->known_width) h->known_width = c.n_phys;
    if (c.done) h->finished = true;
    return SKB_OK;
}

// A snapshot of the control block that an earlier step() left in flight: absorb it if it has
// arrived (wait == false: only look), so that device-side errors surface and the launch width
// follows the survivors without any call ever blocking.
static skb_status poll_snapshot(skb_batch *h, bool wait)
{
    if (!h->snap_pending) return SKB_OK;
    cudaError_t e = wait ? cudaEventSynchronize(h->ev[h->snap_idx]) : cudaEventQuery(h->ev[h->snap_idx]);
    if (e == cudaErrorNotReady) return SKB_OK;
    h->snap_pending = false;
    if (e != cudaSuccess) return cuda_fail(h, e, "snapshot");
    return absorb(h, h->h_ctl[h->snap_idx]);
}

extern "C" skb_status sinkhorn_batch_step(skb_batch *h, int cycles)
{
    NvtxRange nvtx_range("skb:step");
    if (!h) return SKB_ERR_NULL;
    if (cycles < 0) return fail(h, SKB_ERR_VALUE, "cycles must be >= 0");
    skb_status st = poll_snapshot(h, false);
    if (st != SKB_OK) return st;
    cudaError_t e;
    if (cycles_in_one_launch(h)) {
        for (int left = cycles; left > 0 && !h->finished; left -= MAX_CYCLES_IN_LAUNCH)
            enqueue_cycles_launch(h, left < MAX_CYCLES_IN_LAUNCH ? left : MAX_CYCLES_IN_LAUNCH);
    } else {
        for (int i = 0; i < cycles && !h->finished; ++i) {
            enqueue_cycle(h);
            if (h->profiling && h->pev_used + PHASE_EVENTS_PER_CYCLE > (int)h->pev.size() &&
                (e = harvest_phases(h)) != cudaSuccess) return cuda_fail(h, e, "step (phase timing)");
        }
    }
    if (!h->snap_pending && cycles > 0) {
        h->snap_idx ^= 1;
        if ((e = cudaMemcpyAsync(&h->h_ctl[h->snap_idx], h->dev.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost, h->stream)) != cudaSuccess ||
            (e = cudaEventRecord(h->ev[h->snap_idx], h->stream)) != cudaSuccess) return cuda_fail(h, e, "step");
        h->snap_pending = true;
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e, "step");
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_drain(skb_batch *h, int *cycles_run)
{
    NvtxRange nvtx_range("skb:drain");
    if (!h) return SKB_ERR_NULL;
    cudaError_t e;
    {
        skb_status st0 = poll_snapshot(h, true);
        if (st0 != SKB_OK) { cudaStreamSynchronize(h->stream); return st0; }
    }
    int chunk = 2, snap = 0, rounds = 0;
    bool have_prev = false;
    // every lane is retired by the audit that follows cycle max_iter; STATIC needs one more pass
    const long long hard_cap = (long long)h->cfg.max_iter + 4;
    while (!h->finished) {
        const bool multi = cycles_in_one_launch(h);      // may become true as the batch narrows
        const int chunk_max = multi ? 32 : 16;
        NvtxRange nvtx_chunk(multi ? "skb:chunk (cycles in one launch)" : "skb:chunk (launch per leg)");
        if (multi) enqueue_cycles_launch(h, chunk);
        else for (int i = 0; i < chunk; ++i) enqueue_cycle(h);
        if (h->profiling && (e = harvest_phases(h)) != cudaSuccess) return cuda_fail(h, e, "drain (phase timing)");
        if ((e = cudaMemcpyAsync(&h->h_ctl[snap], h->dev.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost, h->stream)) != cudaSuccess)
            return cuda_fail(h, e, "drain");
        if ((e = cudaEventRecord(h->ev[snap], h->stream)) != cudaSuccess) return cuda_fail(h, e, "drain");
        if (have_prev) {
            if ((e = cudaEventSynchronize(h->ev[snap ^ 1])) != cudaSuccess) return cuda_fail(h, e, "drain");
            skb_status st = absorb(h, h->h_ctl[snap ^ 1]);
            if (st != SKB_OK) { cudaStreamSynchronize(h->stream); return st; }
        }
        have_prev = true;
        snap ^= 1;
        // grow the chunk every other round: cycles enqueued past completion are empty launches that
        // still have to drain, which matters for batches that finish within a dozen cycles
        if (chunk < chunk_max && (++rounds & 1) == 0) chunk *= 2;
        if (h->enqueued - h->enqueued_at_refill > hard_cap + 64) break;
    }
    if ((e = cudaStreamSynchronize(h->stream)) != cudaSuccess) return cuda_fail(h, e, "drain");
    if ((e = cudaMemcpy(&h->h_ctl[0], h->dev.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost)) != cudaSuccess)
        return cuda_fail(h, e, "drain");
    skb_status st = absorb(h, h->h_ctl[0]);
    if (st != SKB_OK) return st;
    if (!h->finished) return fail(h, SKB_ERR_STATE, "drain ended with lanes still running");
    if (cycles_run) *cycles_run = h->h_ctl[0].cycle;
    return SKB_OK;
}

static skb_status read_ctl(skb_batch *h, Ctl *c)
{
    cudaError_t e;
    if ((e = cudaStreamSynchronize(h->stream)) != cudaSuccess) return cuda_fail(h, e, "sync");
    if ((e = cudaMemcpy(&h->h_ctl[0], h->dev.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost)) != cudaSuccess)
        return cuda_fail(h, e, "read control block");
    *c = h->h_ctl[0];
    return absorb(h, *c);
}

extern "C" skb_status sinkhorn_batch_active(skb_batch *h, int *n_active)
{
    if (!h || !n_active) return SKB_ERR_NULL;
    Ctl c;
    skb_status st = read_ctl(h, &c);
    if (st != SKB_OK) return st;
    *n_active = c.done ? 0 : (h->cfg.mode == SKB_STATIC ? h->cfg.W : c.n_running);
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_potentials(skb_batch *h, float *f, float *g)
{
    if (!h) return SKB_ERR_NULL;
    launch_gather(h->dev, f, g, false, h->stream);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : cuda_fail(h, e, "potentials");
}

extern "C" skb_status sinkhorn_batch_potentials_f64(skb_batch *h, double *f, double *g)
{
    if (!h) return SKB_ERR_NULL;
    launch_gather(h->dev, f, g, true, h->stream);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : cuda_fail(h, e, "potentials");
}

extern "C" skb_status sinkhorn_batch_depths(skb_batch *h, int *depth, int *lane_status)
{
    if (!h) return SKB_ERR_NULL;
    launch_gather_small(h->dev, depth, lane_status, nullptr, nullptr, h->stream);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : cuda_fail(h, e, "depths");
}

extern "C" skb_status sinkhorn_batch_residuals(skb_batch *h, float *r_row, float *r_col)
{
    if (!h) return SKB_ERR_NULL;
    launch_gather_small(h->dev, nullptr, nullptr, r_row, r_col, h->stream);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : cuda_fail(h, e, "residuals");
}

extern "C" skb_status sinkhorn_batch_apply_plan(skb_batch *h, const void *x, const void *y, const float *eps,
                                                const float *v, int dv, float *out)
{
    if (!h) return SKB_ERR_NULL;
    if (!x || !y || !eps || !v || !out) return fail(h, SKB_ERR_NULL, "x, y, eps, v and out are required");
    if (dv < 1 || dv > 16) return fail(h, SKB_ERR_SHAPE, "dv must be between 1 and 16");
    if (h->lanes_used > h->cfg.W) return fail(h, SKB_ERR_STATE, "not available for batches whose lanes were replaced (the inputs of all lanes are not in one array)");
    Ctl c;
    skb_status st = read_ctl(h, &c);
    if (st != SKB_OK) return st;
    if (!c.done) return fail(h, SKB_ERR_STATE, "the plan is applied once every lane has finished (drain first)");
    launch_apply_plan(h->dev, x, y, eps, v, dv, out, h->cfg.W, h->stream);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : cuda_fail(h, e, "apply_plan");
}

extern "C" skb_status sinkhorn_batch_last_audit(skb_batch *h, float *r_row, float *r_col, int *flagged)
{
    if (!h) return SKB_ERR_NULL;
    if (cycles_in_one_launch(h)) return fail(h, SKB_ERR_STATE, "per-audit values are kept by the one-launch-per-leg path only (MASKED, STATIC, tensor or profiled batches)");
    launch_gather_audit(h->dev, r_row, r_col, flagged, h->stream);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : cuda_fail(h, e, "last_audit");
}

extern "C" skb_status sinkhorn_batch_stats(skb_batch *h, long long *slots, int *cycles, int *widths,
                                           int widths_cap, long long *pair_terms, float *phase_ms)
{
    if (!h) return SKB_ERR_NULL;
    Ctl c;
    skb_status st = read_ctl(h, &c);
    if (st != SKB_OK) return st;
    if (h->profiling) {
        cudaError_t e = harvest_phases(h);
        if (e != cudaSuccess) return cuda_fail(h, e, "stats (phase timing)");
    }
    if (phase_ms) for (int i = 0; i < SKB_N_PHASES; ++i) phase_ms[i] = h->phase_ms[i];
    if (slots) *slots = c.slots;
    if (cycles) *cycles = c.cycle;
    if (pair_terms) *pair_terms = c.pair_terms;
    if (widths && widths_cap > 0) {
        int k = c.cycle < widths_cap ? c.cycle : widths_cap;
        if (k > h->dev.widths_cap) k = h->dev.widths_cap;
        cudaError_t e = cudaMemcpy(widths, h->dev.widths, (size_t)k * sizeof(int), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return cuda_fail(h, e, "stats");
    }
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_cycle_trace(skb_batch *h, float *update_ms, int cap, int *count)
{
    if (!h || !count) return SKB_ERR_NULL;
    if (h->profiling) {
        cudaError_t e = cudaStreamSynchronize(h->stream);
        if (e == cudaSuccess) e = harvest_phases(h);
        if (e != cudaSuccess) return cuda_fail(h, e, "cycle_trace");
    }
    const int n = (int)h->cycle_update_ms.size();
    *count = n;
    if (update_ms) for (int i = 0; i < n && i < cap; ++i) update_ms[i] = h->cycle_update_ms[i];
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_arithmetic(skb_batch *h, int *compute)
{
    if (!h || !compute) return SKB_ERR_NULL;
    *compute = h->tensor ? SKB_COMPUTE_TENSOR : (!h->var->f64 ? SKB_COMPUTE_F32 : (h->var->xf ? SKB_COMPUTE_MIXED : SKB_COMPUTE_F64));
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_check_guards(skb_batch *h, int *first_bad)
{
    if (!h || !first_bad) return SKB_ERR_NULL;
    *first_bad = -1;
    cudaError_t e = cudaMemsetAsync(h->dev.guard_bad, 0xFF, sizeof(int), h->stream);      // atomicMin target: all ones
    if (e != cudaSuccess) return cuda_fail(h, e, "check_guards");
    launch_guard_strips(h->cfg.workspace, h->guards, false, h->dev.guard_bad, h->stream);
    h->launches += 1;
    unsigned found = 0xFFFFFFFFu;
    if ((e = cudaGetLastError()) != cudaSuccess ||
        (e = cudaMemcpyAsync(&found, h->dev.guard_bad, sizeof(int), cudaMemcpyDeviceToHost, h->stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(h->stream)) != cudaSuccess)
        return cuda_fail(h, e, "check_guards");
    if (found != 0xFFFFFFFFu) *first_bad = (int)found - 1;
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_selftest_bounded_wait(int *out3, float budget_ms, void *stream)
{
    if (!out3) return SKB_ERR_NULL;
    if (!(budget_ms > 0.0f) || budget_ms > 2000.0f) return fail(nullptr, SKB_ERR_VALUE, "budget must be in (0, 2000] ms");
    launch_wait_probe(out3, (long long)(budget_ms * 2.0e6f), (cudaStream_t)stream);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SKB_OK : cuda_fail(nullptr, e, "selftest");
}

extern "C" skb_status sinkhorn_batch_launch_count(skb_batch *h, long long *launches)
{
    if (!h || !launches) return SKB_ERR_NULL;
    *launches = h->launches;
    return SKB_OK;
}

extern "C" skb_status sinkhorn_batch_profile_update(skb_batch *h, int leg, int reps, float *ms_per_launch)
{
    if (!h || !ms_per_launch) return SKB_ERR_NULL;
    if ((leg != LEG_F && leg != LEG_G) || reps < 1) return fail(h, SKB_ERR_VALUE, "leg must be 0 or 1 and reps >= 1");
    Ctl now;
    skb_status st0 = read_ctl(h, &now);
    if (st0 != SKB_OK) return st0;
    if (now.done || now.static_final) return fail(h, SKB_ERR_STATE, "no lane is running: an update launch would return at once");
    cudaEvent_t a, b;
    cudaError_t e;
    if ((e = cudaEventCreate(&a)) != cudaSuccess) return cuda_fail(h, e, "profile");
    if ((e = cudaEventCreate(&b)) != cudaSuccess) { cudaEventDestroy(a); return cuda_fail(h, e, "profile"); }
    // dry-run launches: the leg does all of its pair work and its row epilogue but stores no potential
    // and adds no residual term, so the batch's state is exactly what it was
    const Dev saved = h->dev;
    h->dev.dry_run = 1;
    launch_leg(h, leg, h->known_width);          // warm-up
    cudaEventRecord(a, h->stream);
    for (int i = 0; i < reps; ++i) launch_leg(h, leg, h->known_width);
    cudaEventRecord(b, h->stream);
    h->dev = saved;
    e = cudaEventSynchronize(b);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
    cudaEventDestroy(a); cudaEventDestroy(b);
    h->launches += reps + 1;
    if (e != cudaSuccess) return cuda_fail(h, e, "profile");
    *ms_per_launch = ms / (float)reps;
    return SKB_OK;
}

struct HostStage { size_t x, y, a, b, eps, f, g, depth, status, rrow, rcol, end; };

static HostStage host_stage(const skb_config *c, size_t base)
{
    HostStage s;
    size_t off = align_up(base, 256);
    auto take = [&](size_t b) { size_t o = off; off += align_up(b, 256); return o; };
    const size_t W = c->W, n = c->n, m = c->m, d = c->d, es = c->xy_dtype == SKB_BF16 ? 2 : 4;
    s.x = take(W * n * d * es); s.y = take(W * m * d * es);
    s.a = take(W * n * 4); s.b = take(W * m * 4); s.eps = take(W * 4);
    s.f = take(W * n * 4); s.g = take(W * m * 4);
    s.depth = take(W * 4); s.status = take(W * 4); s.rrow = take(W * 4); s.rcol = take(W * 4);
    s.end = off;
    return s;
}

extern "C" size_t sinkhorn_batch_host_workspace_bytes(const skb_config *cfg)
{
    const size_t core = sinkhorn_batch_workspace_bytes(cfg);
    if (core == 0) return 0;
    return host_stage(cfg, core).end;
}

extern "C" skb_status sinkhorn_batch_solve_host(const void *x, const void *y, const float *a, const float *b,
                                                const float *eps, float tol, const skb_config *cfg,
                                                float *f, float *g, int *depth, int *lane_status,
                                                float *r_row, float *r_col, long long *slots, int *cycles)
{
    if (!x || !y || !a || !b || !eps || !cfg) return fail(nullptr, SKB_ERR_NULL, "x, y, a, b, eps and cfg are required");
    const size_t core = sinkhorn_batch_workspace_bytes(cfg);
    if (core == 0) return fail(nullptr, SKB_ERR_SHAPE, "configuration rejected");
    const HostStage s = host_stage(cfg, core);
    if (!cfg->workspace || cfg->workspace_bytes < s.end) return fail(nullptr, SKB_ERR_WORKSPACE, "workspace too small for the host-buffer call");
    char *base = (char *)cfg->workspace;
    cudaStream_t st = (cudaStream_t)cfg->stream;
    const size_t W = cfg->W, n = cfg->n, m = cfg->m, d = cfg->d, es = cfg->xy_dtype == SKB_BF16 ? 2 : 4;
    cudaError_t e;
    if ((e = cudaMemcpyAsync(base + s.x, x, W * n * d * es, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(base + s.y, y, W * m * d * es, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(base + s.a, a, W * n * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(base + s.b, b, W * m * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(base + s.eps, eps, W * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess)
        return cuda_fail(nullptr, e, "solve_host (copy in)");
    skb_config inner = *cfg;
    inner.workspace_bytes = core;
    skb_batch *h = nullptr;
    skb_status rc = sinkhorn_batch_create(base + s.x, base + s.y, (const float *)(base + s.a), (const float *)(base + s.b),
                                          (const float *)(base + s.eps), tol, &inner, &h);
    if (rc != SKB_OK) return rc;
    int cyc = 0;
    rc = sinkhorn_batch_drain(h, &cyc);
    if (rc == SKB_OK) rc = sinkhorn_batch_potentials(h, f ? (float *)(base + s.f) : nullptr, g ? (float *)(base + s.g) : nullptr);
    if (rc == SKB_OK) rc = sinkhorn_batch_depths(h, (int *)(base + s.depth), (int *)(base + s.status));
    if (rc == SKB_OK) rc = sinkhorn_batch_residuals(h, (float *)(base + s.rrow), (float *)(base + s.rcol));
    if (rc == SKB_OK) {
        e = cudaSuccess;
        if (f) e = cudaMemcpyAsync(f, base + s.f, W * n * 4, cudaMemcpyDeviceToHost, st);
        if (g && e == cudaSuccess) e = cudaMemcpyAsync(g, base + s.g, W * m * 4, cudaMemcpyDeviceToHost, st);
        if (depth && e == cudaSuccess) e = cudaMemcpyAsync(depth, base + s.depth, W * 4, cudaMemcpyDeviceToHost, st);
        if (lane_status && e == cudaSuccess) e = cudaMemcpyAsync(lane_status, base + s.status, W * 4, cudaMemcpyDeviceToHost, st);
        if (r_row && e == cudaSuccess) e = cudaMemcpyAsync(r_row, base + s.rrow, W * 4, cudaMemcpyDeviceToHost, st);
        if (r_col && e == cudaSuccess) e = cudaMemcpyAsync(r_col, base + s.rcol, W * 4, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) rc = cuda_fail(nullptr, e, "solve_host (copy out)");
    }
    if (rc == SKB_OK && (slots || cycles)) rc = sinkhorn_batch_stats(h, slots, cycles, nullptr, 0, nullptr, nullptr);
    if (rc != SKB_OK && h) g_create_err = h->err;
    sinkhorn_batch_destroy(h);
    return rc;
}

extern "C" void sinkhorn_batch_destroy(skb_batch *h)
{
    if (!h) return;
    if (h->stream || h->h_ctl) cudaStreamSynchronize(h->stream);
    for (cudaEvent_t ev : h->pev) if (ev) cudaEventDestroy(ev);
    if (h->h_ctl && h->ev[0] && h->ev[1]) {
        HostRes r; r.pinned = h->h_ctl; r.ev[0] = h->ev[0]; r.ev[1] = h->ev[1]; r.device = h->res_device;
        host_res_put(r);
    } else {
        if (h->ev[0]) cudaEventDestroy(h->ev[0]);
        if (h->ev[1]) cudaEventDestroy(h->ev[1]);
        if (h->h_ctl) cudaFreeHost(h->h_ctl);
    }
    delete h;
}

extern "C" const char *sinkhorn_batch_last_error(const skb_batch *h)
{
    return h ? h->err.c_str() : g_create_err.c_str();
}
