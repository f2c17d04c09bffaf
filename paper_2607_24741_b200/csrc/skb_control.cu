// Set-up, audit planning, retirement/compaction and read-back kernels.
//
//  prep       inputs -> the kernels' layout (scaled dimension-major coordinates, squared
//             norms, log2 weights, cold potentials f = g = 0); validates values.
//  plan       one CTA per audit: turns the per-lane flags into the retire list by a warp
//             ballot / prefix-sum scan, records depth, status and residuals of retirees
//             (completion depth l_t, Eq. 6), pairs every hole left below the new width
//             with a survivor from above it, and advances the counters of Eq. 7.
//  warm       replaces the cold potentials by a caller's proposal (Section "Initialization and
//             repeated couplings"), before the first cycle.
//  emit_move  writes retirees' potentials to the result buffers in the caller's units and
//             moves every slot-indexed array of a paired survivor into the hole it fills
//             (Section "Screen, verify, and compact").  Holes and sources are disjoint slot
//             sets, so the in-place copies cannot race.
//  gather     potentials in original lane order (retired lanes from the result buffers,
//             running lanes from their slots).
#include "skb_device.cuh"
#include "skb_host.h"

namespace skb {

// ---------------------------------------------------------------- prep
// One CTA per lane: joint centroid of the two clouds, the largest scaled squared distance
// from it, and from that the cost form the lane will use.
// Lanes come in as a block of problems: input problem q goes to slot slot0 + q as lane lane0 + q
// (create: slot0 = lane0 = 0, all W; a refill: the first free slot, the next unused lane number).
__global__ void __launch_bounds__(256) lane_stats_kernel(const Dev P, const void *xin, const void *yin, const float *eps,
                                                         const int slot0, const int lane0, const int cycle0)
{
    __shared__ double red[256];
    __shared__ double cen[1024];
    const int q = blockIdx.x, slot = slot0 + q, tid = threadIdx.x;
    const int tot = P.n + P.m;
    for (int k = 0; k < P.d; ++k) {
        double s = 0.0;
        for (int p = tid; p < tot; p += 256) {
            const bool isx = p < P.n;
            const size_t idx = isx ? ((size_t)q * P.n + p) * P.d + k : ((size_t)q * P.m + (p - P.n)) * P.d + k;
            s += (double)load_raw(P, isx ? xin : yin, idx);
        }
        red[tid] = s;
        __syncthreads();
        for (int off = 128; off > 0; off >>= 1) { if (tid < off) red[tid] += red[tid + off]; __syncthreads(); }
        if (tid == 0) cen[k] = red[0] / (double)tot;
        __syncthreads();
    }
    double mxr = 0.0;
    for (int p = tid; p < tot; p += 256) {
        const bool isx = p < P.n;
        const size_t base = isx ? ((size_t)q * P.n + p) * P.d : ((size_t)q * P.m + (p - P.n)) * P.d;
        double r2 = 0.0;
        for (int k = 0; k < P.d; ++k) { const double v = (double)load_raw(P, isx ? xin : yin, base + k) - cen[k]; r2 += v * v; }
        mxr = fmax(mxr, r2);
    }
    red[tid] = mxr;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) { if (tid < off) red[tid] = fmax(red[tid], red[tid + off]); __syncthreads(); }
    for (int k = tid; k < P.DP; k += 256) P.center[(size_t)slot * P.DP + k] = k < P.d ? cen[k] : 0.0;
    if (tid == 0) {
        const double e = (double)eps[q];
        const bool eps_ok = (e > 0.0) && isfinite(e);
        const double s = eps_ok ? 1.4426950408889634 / e : 1.0;
        if (!eps_ok) atomicOr(&P.ctl->error, ERR_VALUE);
        P.scale[slot] = s;
        P.lane_id[slot] = lane0 + q;
        P.start[slot] = cycle0;
        // whatever an earlier lane left in the slot
        P.nonfinite[slot] = 0; P.state[slot] = 0; P.flag[slot] = 0; P.verdict[slot] = 0;
        P.rsum_row[slot] = 0ull; P.rsum_col[slot] = 0ull; P.rsum_row64[slot] = 0ull; P.esc[slot] = 0;
        P.ret_at[slot] = 0; P.n_checks[slot] = 0;
        int form = P.cost_form == 1 ? FORM_DOT : (P.cost_form == 2 ? FORM_DIFF : (s * red[0] > P.form_threshold ? FORM_DIFF : FORM_DOT));
        P.form[slot] = form;
        atomicMax(&P.ctl->max_radius_bits, (unsigned long long)__double_as_longlong(eps_ok ? s * red[0] : 0.0));
    }
}

template <typename T>
__global__ void prep_kernel(const Dev P, const void *xin, const void *yin, const float *a, const float *b, const int slot0)
{
    const int q = blockIdx.y, slot = slot0 + q;
    const int side = blockIdx.z;                     // 0: x / a, 1: y / b
    const int npts = side ? P.m : P.n, pp = side ? P.mp : P.np;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= pp) return;
    const double s = P.scale[slot];
    const int form = (sizeof(T) == 8) ? (int)FORM_DOT : P.form[slot];
    T *crd = reinterpret_cast<T *>(side ? P.ys : P.xs) + (size_t)slot * P.DP * pp;
    const size_t o = (size_t)slot * pp + i;
    T *hi0 = side ? reinterpret_cast<T *>(P.gt) : reinterpret_cast<T *>(P.ft[0]);
    T *lo0 = side ? reinterpret_cast<T *>(P.gl) : reinterpret_cast<T *>(P.fl[0]);
    double *sq = side ? P.sqy : P.sqx, *lw = side ? P.lb2 : P.la2, *wt = side ? P.wb : P.wa;
    T hi, lo = T(0);
    if (i >= npts) {                                  // padding points
        if (!P.tensor) for (int k = 0; k < P.DP; ++k) crd[(size_t)k * pp + i] = T(0);
        hi = T(NEG_BIG);
        sq[o] = 0.0; lw[o] = 0.0; wt[o] = 0.0;
    } else {
        // tensor-core path: raw coordinates feed the MMA, the scale 2s is applied to its result
        const double sc = P.tensor ? sqrt(2.0 * s) : sqrt(form == FORM_DOT ? 2.0 * s : s);
        const size_t ibase = ((size_t)q * npts + i) * P.d;
        const double *cen = P.center + (size_t)slot * P.DP;
        double nrm = 0.0;
        bool ok = true;
        for (int k = 0; k < P.DP; ++k) {
            T v = T(0);
            if (k < P.d) {
                const float raw = load_raw(P, side ? yin : xin, ibase + k);
                ok = ok && isfinite(raw);
                v = P.tensor ? (T)0 : (T)(sc * ((double)raw - cen[k]));
                if (P.tensor) nrm += (sc * (double)raw) * (sc * (double)raw);
            }
            if (!P.tensor) crd[(size_t)k * pp + i] = v;
            nrm += (double)v * (double)v;
        }
        nrm = form == FORM_DOT ? 0.5 * nrm : 0.0;
        const float w = (side ? b : a)[(size_t)q * npts + i];
        ok = ok && (w > 0.0f) && isfinite(w);
        if (!ok) atomicOr(&P.ctl->error, ERR_VALUE);
        sq[o] = nrm;
        lw[o] = ok ? log2((double)w) : 0.0;
        wt[o] = ok ? (double)w : 0.0;
        hi = (T)(-nrm);                                // cold start: phi = gam = 0
    }
    hi0[o] = hi; lo0[o] = lo;
    if (!side) {
        reinterpret_cast<T *>(P.ft[1])[o] = hi; reinterpret_cast<T *>(P.fl[1])[o] = lo;
        P.phi[0][o] = 0.0; P.phi[1][o] = 0.0;
    } else {
        P.gam[o] = 0.0;
    }
}

// Warm proposal: potentials in the caller's units -> the kernels' representation of both buffers
// (same formulas as the cold start in prep_kernel, with phi = s f0 and gam = s g0 instead of 0).
// Runs before the first cycle, when slot t still holds lane t.
template <typename T>
__global__ void warm_kernel(const Dev P, const double *f0, const double *g0)
{
    const int slot = blockIdx.y, side = blockIdx.z;
    const int npts = side ? P.m : P.n, pp = side ? P.mp : P.np;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= npts) return;
    const double *src = side ? g0 : f0;
    if (!src) return;
    const double v = src[(size_t)slot * npts + i];
    if (!isfinite(v)) { atomicOr(&P.ctl->error, ERR_VALUE); return; }
    const int form = (sizeof(T) == 8) ? (int)FORM_DOT : P.form[slot];
    const size_t o = (size_t)slot * pp + i;
    const double pot = P.scale[slot] * v;
    T hi, lo;
    if (form == FORM_DOT) { hi = (T)(pot - (side ? P.sqy : P.sqx)[o]); lo = T(0); }
    else { hi = (T)pot; lo = (T)(pot - (double)hi); }
    if (!side) {
        P.phi[0][o] = pot; P.phi[1][o] = pot;
        reinterpret_cast<T *>(P.ft[0])[o] = hi; reinterpret_cast<T *>(P.ft[1])[o] = hi;
        reinterpret_cast<T *>(P.fl[0])[o] = lo; reinterpret_cast<T *>(P.fl[1])[o] = lo;
    } else {
        P.gam[o] = pot;
        reinterpret_cast<T *>(P.gt)[o] = hi; reinterpret_cast<T *>(P.gl)[o] = lo;
    }
}

// ---------------------------------------------------------------- plan
constexpr int PLAN_THREADS = 1024;   // upper bound; the launch sizes the block to the width

// exclusive prefix sums of up to three 0/1 flags over the block, by warp ballot + popc
__device__ __forceinline__ void block_scan3(int f0, int f1, int f2, int (&ex)[3], int (&tot)[3], int (*wsum)[3])
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned lt = (1u << lane) - 1u;
    const unsigned b0 = __ballot_sync(0xffffffffu, f0), b1 = __ballot_sync(0xffffffffu, f1),
                   b2 = __ballot_sync(0xffffffffu, f2);
    ex[0] = __popc(b0 & lt); ex[1] = __popc(b1 & lt); ex[2] = __popc(b2 & lt);
    __syncthreads();
    if (lane == 0) { wsum[warp][0] = __popc(b0); wsum[warp][1] = __popc(b1); wsum[warp][2] = __popc(b2); }
    __syncthreads();
    int run[3] = {0, 0, 0};
    const int nwarp = blockDim.x >> 5;
    for (int w = 0; w < nwarp; ++w) {
        if (w == warp) { ex[0] += run[0]; ex[1] += run[1]; ex[2] += run[2]; }
        run[0] += wsum[w][0]; run[1] += wsum[w][1]; run[2] += wsum[w][2];
    }
    tot[0] = run[0]; tot[1] = run[1]; tot[2] = run[2];
}

template <typename T>
__device__ __forceinline__ void emit_move_one(const Dev &P, const Ctl &c, const int r, const int tid, const int nth);

// FUSE: the same block also emits and moves the lanes it retires (see launch_plan).
template <typename T, bool FUSE>
__global__ void __launch_bounds__(PLAN_THREADS) plan_kernel(const Dev P)
{
    __shared__ int wsum[PLAN_THREADS / 32][3];
    pdl_enter();
    Ctl c = *P.ctl;
    const int tid = threadIdx.x, NT = blockDim.x;
    if (c.done) { if (tid == 0) P.ctl->n_retire = 0; return; }
    const int k = c.cycle;                           // cycles completed by the audited state
    const int A = c.n_phys;
    // a lane has used up its cycles when ITS OWN count reaches max_iter (lanes that replaced finished
    // ones came in later; everywhere else start is 0)
    auto at_limit = [&](int s) { return k - P.start[s] >= P.max_iter; };

    if (P.mode == MODE_STATIC && c.static_final) {   // emit every lane at the common boundary
        for (int s = tid; s < P.W; s += NT) {
            P.ret_slot[s] = s; P.ret_lane[s] = s; P.ret_src[s] = -1; P.ret_scale[s] = P.scale[s];
            // the closing column check ran no f-leg: r_row is the last screen's value
            P.res_row[s] = P.rrow[s]; P.res_col[s] = (double)P.rsum_col[s] * (1.0 / RSUM_SCALE);
            P.rsum_col[s] = 0ull;
            if (P.nonfinite[s]) P.status[s] = LANE_NONFINITE;
        }
        if (tid == 0) {
            Ctl *g = P.ctl;
            g->n_retire = FUSE ? 0 : P.W; g->emit_parity = c.parity; g->n_running = 0; g->done = 1;
            g->pair_terms += (long long)P.W * P.n * P.m;      // the final column check
        }
        if (FUSE) {
            __syncthreads();
            Ctl cc = c;
            cc.emit_parity = c.parity;
            for (int r = 0; r < P.W; ++r) emit_move_one<T>(P, cc, r, tid, NT);
        }
        return;
    }

    // which running lanes leave at this audit
    auto decide_vals = [&](bool held, int nf, int fl, int vd, bool limit, int &ret, int &st) {
        ret = 0; st = LANE_RUNNING;
        if (held) return;
        if (nf) { ret = 1; st = LANE_NONFINITE; }
        else if (fl && vd) { ret = 1; st = LANE_DONE; }
        else if (limit) { ret = 1; st = LANE_ITER_LIMIT; }
    };
    auto decide = [&](int s, int &ret, int &st) {
        ret = 0; st = LANE_RUNNING;
        if (s >= A) return;
        const bool held = (P.mode != MODE_ACTIVE) && P.state[s] != 0;   // frozen / already passed
        decide_vals(held, P.nonfinite[s], P.flag[s], P.verdict[s], at_limit(s), ret, st);
    };

    // pass 1.  The legs left each lane's residuals as exact fixed-point sums: turn them into the
    // values, the screen flag and the two-sided verdict (Eq. 5), clear the sums for the next
    // cycle, and count retirees and screen-positive lanes on the way.
    int cnt = 0, nflag = 0;
    for (int s = tid; s < A; s += NT) {
        const int fl = lane_flag(P, c, s) ? 1 : 0;
        const int nf = P.nonfinite[s];
        const bool held = (P.mode != MODE_ACTIVE) && P.state[s] != 0;
        const double rr = lane_row_residual(P, s);
        const double rc = (double)P.rsum_col[s] * (1.0 / RSUM_SCALE);
        const int vd = (!nf && fmax(rr, rc) <= P.tol_stop) ? 1 : 0;
        P.rsum_row[s] = 0ull; P.rsum_col[s] = 0ull; P.rsum_row64[s] = 0ull; P.esc[s] = 0;
        P.rrow[s] = rr; P.rcol[s] = rc;
        P.flag[s] = fl; P.verdict[s] = vd;
        int r, st; decide_vals(held, nf, fl, vd, at_limit(s), r, st);
        cnt += r;
        nflag += fl;
    }
    for (int off = 16; off > 0; off >>= 1) {
        cnt += __shfl_down_sync(0xffffffffu, cnt, off);
        nflag += __shfl_down_sync(0xffffffffu, nflag, off);
    }
    if ((tid & 31) == 0) { wsum[tid >> 5][0] = cnt; wsum[tid >> 5][1] = nflag; }
    __syncthreads();
    int nret = 0, nflagged = 0;
    for (int w = 0; w < (NT >> 5); ++w) { nret += wsum[w][0]; nflagged += wsum[w][1]; }
    __syncthreads();
    const int Anew = (P.mode == MODE_ACTIVE) ? A - nret : A;

    // pass 2: ordered lists (retirees, holes below Anew, survivors at or above Anew);
    // most audits retire nobody and skip it
    int base[3] = {0, 0, 0};
    for (int s0 = 0; s0 < (nret > 0 ? A : 0); s0 += NT) {
        const int s = s0 + tid;
        int r, st; decide(s, r, st);
        const int hole = (P.mode == MODE_ACTIVE) && r && s < Anew;
        const int fill = (P.mode == MODE_ACTIVE) && !r && s >= Anew && s < A;
        int ex[3], tot[3];
        block_scan3(r, hole, fill, ex, tot, wsum);
        if (r) {
            const int idx = base[0] + ex[0];
            const int lane = P.lane_id[s];
            P.ret_slot[idx] = s; P.ret_lane[idx] = lane; P.ret_scale[idx] = P.scale[s];
            P.ret_src[idx] = hole ? -(base[1] + ex[1]) - 2 : -1;      // hole ordinal, resolved below
            if (P.mode != MODE_STATIC || st != LANE_DONE) {            // STATIC keeps residuals for the end
                P.res_row[lane] = P.rrow[s];
                P.res_col[lane] = P.flag[s] ? P.rcol[s] : __longlong_as_double(0x7ff8000000000000LL);
            }
            P.depth[lane] = at_limit(s) && st != LANE_DONE ? P.max_iter : k - P.start[s];
            P.status[lane] = st;
            if (P.mode != MODE_ACTIVE) P.state[s] = 1;
        }
        if (hole) P.hole_list[base[1] + ex[1]] = s;
        if (fill) P.fill_list[base[2] + ex[2]] = s;
        base[0] += tot[0]; base[1] += tot[1]; base[2] += tot[2];
        __syncthreads();
    }
    __threadfence_block();
    __syncthreads();
    const int nholes = base[1];
    // resolve each hole's source, then move the per-slot scalars
    for (int r = tid; r < nret; r += NT) {
        const int code = P.ret_src[r];
        if (code <= -2) P.ret_src[r] = P.fill_list[-(code + 2)];
    }
    __syncthreads();
    for (int h = tid; h < nholes; h += NT) {
        const int dst = P.hole_list[h], src = P.fill_list[h];
        P.lane_id[dst] = P.lane_id[src];
        P.start[dst] = P.start[src];
        P.scale[dst] = P.scale[src];
        P.form[dst] = P.form[src];
        P.nonfinite[dst] = 0;
    }
    if (tid == 0) {
        Ctl *g = P.ctl;
        g->n_retire = (P.mode == MODE_STATIC || FUSE) ? 0 : nret;      // what is left for the emit/move kernel
        g->emit_parity = c.parity;
        // lanes whose pair terms were really evaluated (the early-exit arm skips frozen lanes)
        const int worked = P.early_exit ? c.n_running : A;
        g->pair_terms += (long long)worked * P.n * P.m         // the f-leg that produced this screen
                         + (long long)nflagged * P.n * P.m;    // column checks
        bool go_on;
        if (P.mode == MODE_ACTIVE) {
            g->n_phys = Anew; g->n_running = Anew; go_on = Anew > 0;
        } else if (P.mode == MODE_MASKED) {
            g->n_running = c.n_running - nret; go_on = g->n_running > 0;
        } else {
            g->n_passed = c.n_passed + nret;
            go_on = g->n_passed < P.W;
            if (!go_on) g->static_final = 1;
        }
        if (go_on) {
            const int width = (P.mode == MODE_ACTIVE) ? Anew : (P.early_exit ? g->n_running : P.W);
            g->cycle = k + 1;
            g->parity = c.parity ^ 1;
            g->slots += width;
            g->pair_terms += (long long)width * P.n * P.m;     // the g-leg that completes cycle k+1
            if (k < P.widths_cap) P.widths[k] = width;
        } else if (P.mode != MODE_STATIC) {
            g->done = 1;
        }
    }
    if (FUSE && P.mode != MODE_STATIC && nret > 0) {
        __syncthreads();                                  // the lists and per-slot scalars above are this block's own writes
        Ctl cc = c;
        cc.emit_parity = c.parity;
        for (int r = 0; r < nret; ++r) emit_move_one<T>(P, cc, r, tid, NT);
    }
}

// Planner after a multi-cycle launch (lane_cycles_kernel): the lanes that passed inside the launch
// have written their own depth, status, residuals and potentials; what is left is the accounting of
// Eq. 6-8 for all `K` cycles of the launch at once - widths A_k, slots, pair terms - the pairing of
// holes below the new width with survivors from above it, and the advance of the control block.
template <typename T, bool FUSE>
__global__ void __launch_bounds__(PLAN_THREADS) plan_cycles_kernel(const Dev P, const int K)
{
    __shared__ int wsum[PLAN_THREADS / 32][3];
    __shared__ int left_at[MAX_CYCLES_IN_LAUNCH];   // lanes that left at the audit of the state after k0 + j cycles
    __shared__ int checks_s;
    pdl_enter();
    const Ctl c = *P.ctl;
    const int tid = threadIdx.x, NT = blockDim.x;
    if (c.done) { if (tid == 0) P.ctl->n_retire = 0; return; }
    const int k0 = c.cycle, A = c.n_phys;
    for (int j = tid; j < K; j += NT) left_at[j] = 0;
    if (tid == 0) checks_s = 0;
    __syncthreads();
    int nchk = 0;
    for (int s = tid; s < A; s += NT) {
        const int r = P.ret_at[s];
        if (r > 0) atomicAdd(&left_at[r - 1 - k0], 1);
        nchk += P.n_checks[s];
        P.rsum_row[s] = 0ull; P.rsum_col[s] = 0ull;      // between launches the residual sums are zero
        P.rsum_row64[s] = 0ull; P.esc[s] = 0;
    }
    for (int off = 16; off > 0; off >>= 1) nchk += __shfl_down_sync(0xffffffffu, nchk, off);
    if ((tid & 31) == 0 && nchk) atomicAdd(&checks_s, nchk);
    __syncthreads();
    int nret = 0;
    for (int j = 0; j < K; ++j) nret += left_at[j];
    const int Anew = A - nret;
    const int parity_new = c.parity ^ (K & 1);       // survivors ran all K cycles
    // ordered lists: holes below the new width, survivors at or above it
    int base[3] = {0, 0, 0};
    for (int s0 = 0; s0 < (nret > 0 ? A : 0); s0 += NT) {
        const int s = s0 + tid;
        const int r = (s < A && P.ret_at[s] > 0) ? 1 : 0;
        const int hole = r && s < Anew;
        const int fill = (s < A) && !r && s >= Anew;
        int ex[3], tot[3];
        block_scan3(r, hole, fill, ex, tot, wsum);
        if (hole) P.hole_list[base[1] + ex[1]] = s;
        if (fill) P.fill_list[base[2] + ex[2]] = s;
        base[0] += tot[0]; base[1] += tot[1]; base[2] += tot[2];
        __syncthreads();
    }
    __threadfence_block();
    __syncthreads();
    const int nholes = base[1];
    for (int h = tid; h < nholes; h += NT) {
        const int dst = P.hole_list[h], src = P.fill_list[h];
        P.ret_slot[h] = dst; P.ret_lane[h] = -1; P.ret_src[h] = src; P.ret_scale[h] = 1.0;   // move only
        P.lane_id[dst] = P.lane_id[src];
        P.start[dst] = P.start[src];
        P.scale[dst] = P.scale[src];
        P.form[dst] = P.form[src];
        P.nonfinite[dst] = 0;
    }
    for (int s = tid; s < A; s += NT) { P.ret_at[s] = 0; P.n_checks[s] = 0; }
    if (tid == 0) {
        Ctl *g = P.ctl;
        const long long nm = (long long)P.n * P.m;
        long long slots = 0, terms = (long long)checks_s * nm;
        int w = A, ran = 0;
        for (int j = 0; j < K; ++j) {
            terms += (long long)w * nm;              // the f-leg whose epilogue screened the state after k0 + j cycles
            w -= left_at[j];
            if (w == 0) break;
            if (k0 + j < P.widths_cap) P.widths[k0 + j] = w;      // cycle k0 + j + 1 ran at width w
            slots += w;
            terms += (long long)w * nm;              // its g-leg
            ++ran;
        }
        g->cycle = k0 + ran;
        g->parity = parity_new;
        g->emit_parity = parity_new ^ 1;             // the move copies the OTHER buffer: the survivors' current row potentials
        g->n_phys = Anew; g->n_running = Anew;
        g->n_retire = FUSE ? 0 : nholes;
        g->slots += slots;
        g->pair_terms += terms;
        if (Anew == 0) g->done = 1;
    }
    if (FUSE && nholes > 0) {
        __syncthreads();
        Ctl cc = c;
        cc.emit_parity = parity_new ^ 1;
        for (int r = 0; r < nholes; ++r) emit_move_one<T>(P, cc, r, tid, NT);
    }
}

// ---------------------------------------------------------------- emit + move
template <typename T>
__global__ void __launch_bounds__(256) emit_move_kernel(const Dev P)
{
    pdl_enter();
    const Ctl c = *P.ctl;
    const int nret = c.n_retire;
    if (nret <= 0) return;
    // The launch's blocks are dealt out among the retirees of this audit (usually one or two): a move
    // is a plain copy of up to a few MB and should have the whole machine's loads in flight.
    const int nb = gridDim.x, b = blockIdx.x;
    const int per = nb / nret;
    if (per >= 1) {
        const int r = b / per;
        if (r < nret) emit_move_one<T>(P, c, r, (b % per) * blockDim.x + threadIdx.x, per * blockDim.x);
    } else {
        for (int r = b; r < nret; r += nb) emit_move_one<T>(P, c, r, threadIdx.x, blockDim.x);
    }
}

// Retiree r of the list: `nth` threads (this one is number `tid`) write its outputs and, if its slot
// is a hole below the new width, copy the paired survivor's state into it.
template <typename T>
__device__ __forceinline__ void emit_move_one(const Dev &P, const Ctl &c, const int r, const int tid, const int nth)
{
    const int slot = P.ret_slot[r], lane = P.ret_lane[r], src = P.ret_src[r];
    const double inv_s = 1.0 / P.ret_scale[r];
    const int ep = c.emit_parity;
    // emit: potentials of the audited state in the caller's units (f = phi / s); lane < 0: the lane
    // in the hole wrote its own outputs when it left (multi-cycle launches), only the move is left
    if (lane >= 0)
        for (int i = tid; i < P.n; i += nth)
            P.f_out[(size_t)lane * P.n + i] = P.phi[ep][(size_t)slot * P.np + i] * inv_s;
    for (int j = tid; j < P.m; j += nth) {
        // the hole's own g is read before the survivor's g is copied over it (same thread)
        if (lane >= 0) P.g_out[(size_t)lane * P.m + j] = P.gam[(size_t)slot * P.mp + j] * inv_s;
        if (src >= 0) P.gam[(size_t)slot * P.mp + j] = P.gam[(size_t)src * P.mp + j];
    }
    if (tid == 0 && lane >= 0) P.emitted[lane] = 1;
    if (src < 0) return;
    // Move the survivor in slot `src` into the hole `slot`: all of its slot-indexed arrays as ONE list
    // of 16-byte vectors, so that a thread's loads in flight span arrays (array after array, each
    // with its own loop, cost one DRAM round trip per array: ~15 us for any lane size).
    __shared__ const uint4 *seg_src[16];
    __shared__ uint4 *seg_dst[16];
    __shared__ unsigned seg_end[16];          // running total of vectors up to and including the segment
    __shared__ int seg_n;
    __syncthreads();                          // the table may still be in use by this block's previous retiree
    if (threadIdx.x == 0) {
        int ns = 0;
        unsigned run = 0;
        auto add = [&](void *base, size_t bytes_per_lane) {
            if (!base || bytes_per_lane == 0) return;
            seg_src[ns] = reinterpret_cast<const uint4 *>((const char *)base + (size_t)src * bytes_per_lane);
            seg_dst[ns] = reinterpret_cast<uint4 *>((char *)base + (size_t)slot * bytes_per_lane);
            run += (unsigned)(bytes_per_lane / 16);
            seg_end[ns++] = run;
        };
        const int np_ = ep ^ 1;   // buffer that holds the survivors' current row potentials
        if (P.tensor) {
            add(P.xb, (size_t)((P.n + 127) / 128) * P.d * 256);      // tiled copies: 128-point tiles x d bf16
            add(P.yb, (size_t)((P.m + 127) / 128) * P.d * 256);
        } else {
            add(P.xs, (size_t)P.DP * P.np * sizeof(T));
            add(P.ys, (size_t)P.DP * P.mp * sizeof(T));
        }
        if (P.guard > 0.0) {                                          // raw input copies of the guard band
            add(P.xraw, P.xraw_stride);
            add(P.yraw, P.yraw_stride);
        }
        add(P.sqx, (size_t)P.np * 8); add(P.sqy, (size_t)P.mp * 8);
        add(P.la2, (size_t)P.np * 8); add(P.lb2, (size_t)P.mp * 8);
        add(P.wa, (size_t)P.np * 8); add(P.wb, (size_t)P.mp * 8);
        add(P.phi[np_], (size_t)P.np * 8);
        add(P.ft[np_], (size_t)P.np * sizeof(T));
        add(P.fl[np_], (size_t)P.np * sizeof(T));
        add(P.gt, (size_t)P.mp * sizeof(T));
        add(P.gl, (size_t)P.mp * sizeof(T));
        seg_n = ns;
    }
    __syncthreads();
    const int ns = seg_n;
    const unsigned total = seg_end[ns - 1];
    for (unsigned v = tid; v < total; v += 4u * (unsigned)nth) {       // four loads in flight per thread
        uint4 a[4];
        uint4 *d[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned idx = v + (unsigned)u * (unsigned)nth;
            d[u] = nullptr;
            if (idx < total) {
                int sg = 0;
                while (idx >= seg_end[sg]) ++sg;
                const unsigned off = idx - (sg ? seg_end[sg - 1] : 0u);
                a[u] = seg_src[sg][off];
                d[u] = seg_dst[sg] + off;
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) if (d[u]) *d[u] = a[u];
    }
}

// ---------------------------------------------------------------- gather (read-back)
template <typename O>
__global__ void gather_kernel(const Dev P, O *f, O *g)
{
    const Ctl c = *P.ctl;
    const int y = blockIdx.x;                         // lanes along x: up to twice 65535 of them
    const int tid = blockIdx.y * blockDim.x + threadIdx.x, nth = gridDim.y * blockDim.x;
    if (y < P.L) {                                    // emitted lanes, by lane id
        const int lane = y;
        if (!P.emitted[lane]) return;
        if (f) for (int i = tid; i < P.n; i += nth) f[(size_t)lane * P.n + i] = (O)P.f_out[(size_t)lane * P.n + i];
        if (g) for (int j = tid; j < P.m; j += nth) g[(size_t)lane * P.m + j] = (O)P.g_out[(size_t)lane * P.m + j];
    } else {                                          // lanes still held in a slot
        const int slot = y - P.L;
        if (c.done || slot >= c.n_phys) return;
        if (P.mode == MODE_MASKED && P.state[slot]) return;
        const int lane = P.lane_id[slot];
        if (P.emitted[lane]) return;
        const double inv_s = 1.0 / P.scale[slot];
        if (f) for (int i = tid; i < P.n; i += nth)
            f[(size_t)lane * P.n + i] = (O)(P.phi[c.parity][(size_t)slot * P.np + i] * inv_s);
        if (g) for (int j = tid; j < P.m; j += nth)
            g[(size_t)lane * P.m + j] = (O)(P.gam[(size_t)slot * P.mp + j] * inv_s);
    }
}

__global__ void gather_small_kernel(const Dev P, int *depth, int *status, float *rrow, float *rcol)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= P.L) return;
    if (depth) depth[t] = P.depth[t];
    if (status) status[t] = P.status[t];
    if (rrow) rrow[t] = (float)P.res_row[t];
    if (rcol) rcol[t] = (float)P.res_col[t];
}

// What the most recent audit measured for the lanes still held in a slot (one-launch-per-leg path).
__global__ void gather_audit_kernel(const Dev P, float *rrow, float *rcol, int *flagged)
{
    const Ctl c = *P.ctl;
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= P.W || s >= c.n_phys) return;
    const int lane = P.lane_id[s];
    if (rrow) rrow[lane] = (float)P.rrow[s];
    if (rcol) rcol[lane] = P.flag[s] ? (float)P.rcol[s] : __int_as_float(0x7fc00000);
    if (flagged) flagged[lane] = P.flag[s];
}
void launch_gather_audit(const Dev &P, float *rrow, float *rcol, int *flagged, cudaStream_t st)
{
    gather_audit_kernel<<<(P.W + 255) / 256, 256, 0, st>>>(P, rrow, rcol, flagged);
}

// ---------------------------------------------------------------- plan application
// out[t, i, :] = sum_j pi_ij v[t, j, :] with pi = exp((f + g - C)/eps) from the potentials the batch
// holds for lane t (Eq. 3's plan, never stored): the coupling applied to caller-supplied values, e.g.
// v = y gives a_i times the barycentric image of x_i.  One warp per row, float64 throughout, cost from
// the caller's raw coordinates.  After a g-leg every pi_ij <= b_j <= 1, so the exponentials need no shift.
constexpr int APPLY_MAX_DV = 16;
__global__ void __launch_bounds__(128) apply_plan_kernel(const Dev P, const void *x, const void *y, const float *eps,
                                                         const float *v, const int dv, float *out)
{
    const int lane_t = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * 4 + warp;
    if (i >= P.n || !P.emitted[lane_t]) return;
    const double inv_eps = 1.0 / (double)eps[lane_t];
    const double fi = P.f_out[(size_t)lane_t * P.n + i];
    const double *g = P.g_out + (size_t)lane_t * P.m;
    const size_t xb = ((size_t)lane_t * P.n + i) * P.d;
    double acc[APPLY_MAX_DV];
#pragma unroll
    for (int c = 0; c < APPLY_MAX_DV; ++c) acc[c] = 0.0;
    for (int j = lane; j < P.m; j += 32) {
        const size_t yb = ((size_t)lane_t * P.m + j) * P.d;
        double cst = 0.0;
        for (int k = 0; k < P.d; ++k) {
            const double t = (double)load_raw(P, x, xb + k) - (double)load_raw(P, y, yb + k);
            cst = fma(t, t, cst);
        }
        const double pij = exp((fi + g[j] - cst) * inv_eps);
        const float *vj = v + ((size_t)lane_t * P.m + j) * dv;
#pragma unroll
        for (int c = 0; c < APPLY_MAX_DV; ++c) if (c < dv) acc[c] = fma(pij, (double)vj[c], acc[c]);
    }
#pragma unroll
    for (int c = 0; c < APPLY_MAX_DV; ++c) {
        if (c < dv) {
            double a = acc[c];
            for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
            if (lane == 0) out[((size_t)lane_t * P.n + i) * dv + c] = (float)a;
        }
    }
}
void launch_apply_plan(const Dev &P, const void *x, const void *y, const float *eps, const float *v, int dv, float *out,
                       int lanes, cudaStream_t st)
{
    apply_plan_kernel<<<dim3((P.n + 3) / 4, lanes), 128, 0, st>>>(P, x, y, eps, v, dv, out);
}

// ---------------------------------------------------------------- launchers
void launch_lane_stats(const Dev &P, const void *x, const void *y, const float *eps, int slot0, int lane0, int count,
                       int cycle0, cudaStream_t st)
{
    lane_stats_kernel<<<count, 256, 0, st>>>(P, x, y, eps, slot0, lane0, cycle0);
}
void launch_prep(const Dev &P, const void *x, const void *y, const float *a, const float *b, int slot0, int count, cudaStream_t st)
{
    const int pp = P.np > P.mp ? P.np : P.mp;
    dim3 grid((pp + 127) / 128, count, 2);
    if (P.compute_f64) prep_kernel<double><<<grid, 128, 0, st>>>(P, x, y, a, b, slot0);
    else prep_kernel<float><<<grid, 128, 0, st>>>(P, x, y, a, b, slot0);
}
// New lanes have come in: the control block takes them into the width (between cycles, ACTIVE only).
__global__ void refill_ctl_kernel(const Dev P, const int count)
{
    Ctl *g = P.ctl;
    g->n_phys += count; g->n_running += count; g->done = 0; g->n_retire = 0;
}
void launch_refill_ctl(const Dev &P, int count, cudaStream_t st) { refill_ctl_kernel<<<1, 1, 0, st>>>(P, count); }
void launch_warm(const Dev &P, const double *f0, const double *g0, cudaStream_t st)
{
    const int pp = P.n > P.m ? P.n : P.m;
    dim3 grid((pp + 127) / 128, P.W, 2);
    if (P.compute_f64) warm_kernel<double><<<grid, 128, 0, st>>>(P, f0, g0);
    else warm_kernel<float><<<grid, 128, 0, st>>>(P, f0, g0);
}
// Bytes one retirement can move (a survivor's whole state into the hole) plus what it emits.
static size_t lane_state_bytes(const Dev &P)
{
    const size_t ts = P.compute_f64 ? 8 : 4;
    size_t coords = (size_t)P.DP * (P.np + P.mp) * ts;
    if (P.tensor) coords = ((size_t)((P.n + 127) / 128) + (size_t)((P.m + 127) / 128)) * P.d * 256;
    if (P.guard > 0.0) coords += P.xraw_stride + P.yraw_stride;
    return coords + (size_t)(P.np + P.mp) * (4 * 8 + 2 * ts + 8);
}
// When even the retirement of every lane at once would move little (narrow batches of small
// lanes), the planner's own block emits and moves, and the emit/move kernel is not launched:
// one kernel less in the chain of dependent launches that bounds a narrow cycle.  Same device
// functions either way, so the results do not depend on the choice.
static bool plan_fuses_move(const Dev &P, int width)
{
    const int lanes = (P.mode == MODE_STATIC) ? P.W : (width < 1 ? 1 : width);
    return (size_t)lanes * lane_state_bytes(P) <= ((size_t)512 << 10);
}
int launch_plan(const Dev &P, int width, cudaStream_t st)
{
    int nt = (width + 31) / 32 * 32;
    if (P.mode == MODE_STATIC) nt = (P.W + 31) / 32 * 32;
    const bool fuse = plan_fuses_move(P, width);
    nt = nt < (fuse ? 256 : 128) ? (fuse ? 256 : 128) : (nt > PLAN_THREADS ? PLAN_THREADS : nt);
    if (fuse) {
        if (P.compute_f64) launch_pdl(plan_kernel<double, true>, dim3(1), dim3(nt), 0, st, P);
        else launch_pdl(plan_kernel<float, true>, dim3(1), dim3(nt), 0, st, P);
    } else {
        launch_pdl(plan_kernel<float, false>, dim3(1), dim3(nt), 0, st, P);
    }
    return 1;
}
int launch_plan_cycles(const Dev &P, int width, int cycles, cudaStream_t st)
{
    int nt = (width + 31) / 32 * 32;
    const bool fuse = plan_fuses_move(P, width);
    nt = nt < (fuse ? 256 : 128) ? (fuse ? 256 : 128) : (nt > PLAN_THREADS ? PLAN_THREADS : nt);
    if (fuse) {
        if (P.compute_f64) launch_pdl(plan_cycles_kernel<double, true>, dim3(1), dim3(nt), 0, st, P, cycles);
        else launch_pdl(plan_cycles_kernel<float, true>, dim3(1), dim3(nt), 0, st, P, cycles);
    } else {
        launch_pdl(plan_cycles_kernel<float, false>, dim3(1), dim3(nt), 0, st, P, cycles);
    }
    return 1;
}
int launch_emit_move(const Dev &P, int width, cudaStream_t st)
{
    if (plan_fuses_move(P, width)) return 0;
    if (width < 1) width = 1;
    // one block per 16 KB of a lane's state (four 16-byte vectors per thread and pass), at least one
    // block per lane that could retire at once, at most four blocks per SM
    long long blocks = (long long)((lane_state_bytes(P) + 16383) / 16384);
    if (blocks < (width > 128 ? 128 : width)) blocks = width > 128 ? 128 : width;
    if (blocks > 148 * 4) blocks = 148 * 4;
    if (P.compute_f64) launch_pdl(emit_move_kernel<double>, dim3((unsigned)blocks), dim3(256), 0, st, P);
    else launch_pdl(emit_move_kernel<float>, dim3((unsigned)blocks), dim3(256), 0, st, P);
    return 1;
}
void launch_gather(const Dev &P, void *f, void *g, bool f64, cudaStream_t st)
{
    const int mx = P.n > P.m ? P.n : P.m;
    int gx = (mx + 1023) / 1024; if (gx > 16) gx = 16;
    dim3 grid(P.L + P.W, gx);
    if (f64) gather_kernel<double><<<grid, 256, 0, st>>>(P, (double *)f, (double *)g);
    else gather_kernel<float><<<grid, 256, 0, st>>>(P, (float *)f, (float *)g);
}
void launch_gather_small(const Dev &P, int *depth, int *status, float *rrow, float *rcol, cudaStream_t st)
{
    gather_small_kernel<<<(P.L + 255) / 256, 256, 0, st>>>(P, depth, status, rrow, rcol);
}

// Guard strips: one block per strip, one 32-bit word per thread.  fill = 1 writes the pattern,
// fill = 0 compares and lowers *bad (all ones on entry) to 1 + the index of a damaged strip.
__global__ void __launch_bounds__(GUARD_STRIP_BYTES / 4) guard_strips_kernel(unsigned char *base, const GuardList gl, const int fill, unsigned *bad)
{
    const int strip = blockIdx.x;
    if (strip >= gl.count) return;
    unsigned *w = reinterpret_cast<unsigned *>(base + (size_t)gl.off256[strip] * 256u);
    const unsigned want = 0xA5C3F00Du ^ ((unsigned)strip * 0x9E3779B9u) ^ threadIdx.x;
    if (fill) { w[threadIdx.x] = want; return; }
    if (w[threadIdx.x] != want) atomicMin(bad, (unsigned)strip + 1u);
}
void launch_guard_strips(void *base, const GuardList &gl, bool fill, int *bad, cudaStream_t st)
{
    if (gl.count < 1) return;
    guard_strips_kernel<<<gl.count, GUARD_STRIP_BYTES / 4, 0, st>>>((unsigned char *)base, gl, fill ? 1 : 0, (unsigned *)bad);
}

}  // namespace skb
