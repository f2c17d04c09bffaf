#!/usr/bin/env python
"""Benchmark of the batched shrinking-active-set Sinkhorn hot path on B200.

One "step" = one whole solve of one synthetic batch: create (layout kernels), every cycle
of update / screen / two-sided check / retirement / compaction until all lanes have passed,
results written.  Metric: lane*n*m updates per second, counting one unit per executed
lane-cycle (slot) and point pair, i.e. (sum_k A_k) * n * m / time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload registration] [--mode active]
  python bench.py --impl reference ...     # the float64 CPU oracle on the same workload

The headline workload is `registration` (32 lanes of 8192 x 8192 points, the largest of the five
configurations that one GPU holds).  On one GPU the line also carries a `workloads` object with
all five configurations (active / static / masked time and slots, the dominant kernel against its
rooflines, the phases of the paper's time model, parity against the oracle where the oracle is
cheap enough) and the completion-depth disagreement table of the tolerance sweep.

With N > 1 (launched by torchrun) every rank solves its own replica of the batch: lanes are
independent problems, there is no data-path collective; time is the max over ranks.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "active lane*n*m updates/s (batch time-to-tol 1e-3)"
UNIT = "lane*n*m updates/s"
HEADLINE = "registration"
ALL = ("tiny", "sensor", "feature", "registration", "sweep")

# DRAM bytes (read + write) of ONE full-width f-leg launch of the dominant kernel, from the ncu
# captures summarised in the named files under profiles/ (one launch each; they equal the lanes'
# operands read once).  A kernel whose tiling changes needs a fresh capture: set its entry to None.
NCU_TRAFFIC = {
    "sensor": (20.5e6, "profiles/update_kernel_sensor_registration_sweep.md"),
    "registration": (13.7e6, "profiles/update_kernel_sensor_registration_sweep.md"),
    "sweep": (42.0e6, "profiles/update_kernel_sensor_registration_sweep.md"),
    "feature": (193.3e6, "profiles/update_tc_kernel_feature.md"),
}

# nominal unit counts (148 SMs; per SM and clock: 128 FP32 lanes, 16 special-function lanes,
# 64 FP64 lanes) at the maximum SM clock
SM_COUNT, FP32_LANES, MUFU_LANES, FP64_LANES = 148, 128, 16, 64


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "sm_max_mhz": p.get("sm_max_mhz", 1965.0),
                "bf16_tflops": p.get("bf16_tflops", 1590.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True); self.t.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                pass

    def summary(self):
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 6 and r[2 + i].lower() == "active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def aggregate(dist, local_ms: float, local_units: float):
    """Whole-job numbers from per-rank ones: time = max over ranks, units = sum over ranks."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def make_workload(name):
    from paper_2607_24741_b200 import workloads as wl
    return wl.make(name)


def reference_sample(name, w, cores):
    """Which lanes, and how many cycles of each, one step of the oracle arm runs: a bounded sample of
    the workload (a few seconds of host time), stated in the output."""
    W, n, m, d = w.shape
    if name == "registration":       # one lane-cycle is seconds of one core: one cycle (cost matrix, both legs, audit) per lane
        return np.arange(min(W, cores)), 1, "first cycle only (cost matrix, both legs, audit)"
    if name == "feature":
        return np.arange(min(W, cores)), 12, "first 12 cycles"
    if name == "sweep":
        return np.arange(0, W, max(1, W // (4 * cores)))[:4 * cores], w.max_iter, "every lane to its own depth"
    return np.arange(W), w.max_iter, "every lane to its own depth"


def run_reference(args, rank, world):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of lanes."""
    if rank != 0:
        return
    import oracle
    w = make_workload(args.workload)
    W, n, m, d = w.shape
    cores = os.cpu_count() or 1
    sel, cap, what = reference_sample(args.workload, w, cores)
    times, units, threads = [], 0, 1
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        r = oracle.solve_batch(w.x[sel], w.y[sel], w.a[sel], w.b[sel], w.eps[sel], w.tol, max_iter=cap)
        dt = time.perf_counter() - t0
        threads = r.threads
        if it >= args.warmup:
            times.append(dt)
            units = int(r.depth.sum()) * n * m
    ms = 1e3 * sum(times) / len(times)
    val = units / (ms * 1e-3)
    sample = f"{len(sel)} of {W} lanes, {what}"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "W": W, "n": n, "m": m, "d": d, "tol": w.tol, "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
class Runner:
    """One workload resident on the device, and the measurements made on it."""

    def __init__(self, name, args, dev, tol=None):
        import torch
        from paper_2607_24741_b200 import binding as B
        self.torch, self.B, self.args, self.dev, self.name = torch, B, args, dev, name
        self.w = w = make_workload(name)
        if tol is not None:
            w.tol = tol
        t = lambda v: torch.from_numpy(v).to(dev)
        self.x, self.y = t(w.x), t(w.y)
        if w.xy_dtype == "bf16":
            self.x, self.y = self.x.bfloat16(), self.y.bfloat16()
        self.a, self.b, self.eps = t(w.a), t(w.b), t(w.eps)

    def batch(self, mode, tol=None, **kw):
        w = self.w
        return self.B.SinkhornBatch(self.x, self.y, self.a, self.b, self.eps, w.tol if tol is None else tol, mode=mode,
                                    compute=self.args.compute, max_iter=w.max_iter, **kw)

    def solve(self, mode, collect=False, tol=None, **kw):
        sb = self.batch(mode, tol, **kw)
        sb.drain()
        out = None
        if collect:
            st = sb.stats()
            depth, status = sb.depths()
            out = {"slots": st["slots"], "cycles": st["cycles"], "pair_terms": st["pair_terms"],
                   "launches": sb.launch_count(), "sum_depth": int(depth.sum().item()),
                   "done": int((status == 1).sum().item()), "create_ms": st["phase_ms"]["create"]}
        sb.close()
        return out

    def timed(self, mode, steps, warmup, flush, dist=None, tol=None, **kw):
        """Mean ms per solve over `steps` solves after `warmup`, L2 flushed before each, device-timed."""
        torch = self.torch
        info = None
        for _ in range(warmup):
            info = self.solve(mode, collect=True, tol=tol, **kw)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        total, launches = 0.0, 0
        self.last_step_ms = []
        for _ in range(steps):
            flush.fill_(1)                                             # evict L2 between steps
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            self.solve(mode, tol=tol, **kw)
            e1.record()
            torch.cuda.synchronize()
            self.last_step_ms.append(e0.elapsed_time(e1))
            total += self.last_step_ms[-1]
            launches += info["launches"]
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        return total / steps, info, launches

    def roofline(self, unit_rates=None):
        """Dominant kernel (update kernel, f-leg at full width) against its rooflines."""
        w, args = self.w, self.args
        W, n, m, d = w.shape
        sb = self.batch("static")
        sb.step(2)
        k_ms = sb.profile_update(leg=0, reps=20 if W * n * m < (1 << 30) else 8)
        g_ms = sb.profile_update(leg=1, reps=3)
        arith = sb.arithmetic()
        sb.close()
        pk = peaks()
        f_hz = pk["sm_max_mhz"] * 1e6
        pairs = float(W) * n * m
        # algorithmic work per pair: d FMAs for the cross term, then max, subtract, exponential, add
        # (float64 exponents: d FMAs + max + subtract on the half-rate FP64 pipe)
        wide = arith in ("mixed", "f64")
        inst_per_pair = d + 2 if wide else d + 3
        lanes = FP64_LANES if wide else FP32_LANES
        pipe_peak = SM_COUNT * lanes * f_hz
        mufu_peak = SM_COUNT * MUFU_LANES * f_hz
        achieved_inst = pairs * inst_per_pair / (k_ms * 1e-3)
        achieved_exp = pairs / (k_ms * 1e-3)
        bound_pipe = inst_per_pair / lanes > 1.0 / MUFU_LANES
        traffic, traffic_from = NCU_TRAFFIC.get(self.name, (None, None))
        dtype = {"f32": "f32", "mixed": "f64 exponents / f32 exp", "f64": "f64",
                 "tensor": "bf16 (f32 accumulate, f32 exp)"}[arith]
        if arith == "tensor":
            # the cross term is a dense bf16 contraction: 2*d flops per pair against the measured
            # cuBLAS bf16 burst throughput (kernel timed alone)
            tf = 2.0 * d * pairs / (k_ms * 1e-3) / 1e12
            r = {"bound": "tensor", "kernel": "update_tc_pair_kernel (f-leg, full width)" if d > 256 else "update_tc_kernel (f-leg, full width)",
                 "arithmetic": arith, "achieved": tf, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                 "frac": tf / pk["bf16_tflops"], "exp_frac": achieved_exp / mufu_peak,
                 "ms_per_launch": k_ms, "g_leg_ms_per_launch": g_ms, "pairs_per_launch": pairs,
                 "traffic": traffic, "traffic_source": traffic_from,
                 "peak_source": pk["source"] + " cuBLAS bf16 burst (MEASURED_PEAKS.json)"}
        else:
            r = {"bound": "alu", "kernel": "update_kernel (f-leg, full width)", "arithmetic": arith,
                 "binding_unit": ("fp64 pipe" if wide else "fp32 pipe") if bound_pipe else "special-function unit (ex2)",
                 "achieved": (achieved_inst if bound_pipe else achieved_exp) / 1e12,
                 "peak": (pipe_peak if bound_pipe else mufu_peak) / 1e12,
                 "unit": "T lane-instr/s" if bound_pipe else "T exp/s",
                 "frac": (achieved_inst / pipe_peak) if bound_pipe else (achieved_exp / mufu_peak),
                 "exp_frac": achieved_exp / mufu_peak, "pipe_frac": achieved_inst / pipe_peak,
                 "ms_per_launch": k_ms, "g_leg_ms_per_launch": g_ms, "pairs_per_launch": pairs,
                 "peak_clock_mhz": pk["sm_max_mhz"],
                 "traffic": traffic, "traffic_unit": "bytes per launch (ncu)", "traffic_source": traffic_from,
                 "peak_source": "nominal unit counts x max SM clock"}
            if unit_rates:
                # the same fractions against the rates the unit self-test delivered in this run
                meas_pipe = unit_rates["dfma"] if wide else max(unit_rates["ffma"], unit_rates["ffma2"])
                r["frac_of_measured_unit_rates"] = {"exp": achieved_exp / unit_rates["ex2"],
                                                    "pipe": achieved_inst / meas_pipe}
        return r, dtype, arith

    def phases(self, mode="active"):
        """One profiled solve: the cost record of the paper's time model (Eq. 11)."""
        torch = self.torch
        sb = self.batch(mode)
        sb.set_profiling(True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); sb.drain(); e1.record(); torch.cuda.synchronize()
        st = sb.stats(widths_cap=200000)
        trace = sb.cycle_trace()
        sb.close()
        ph = st["phase_ms"]
        cyc = sum(ph[k] for k in ("f_leg", "column_check", "plan", "emit_move", "g_leg"))
        out = {"ms": {k: round(v, 4) for k, v in ph.items()}, "sum_of_cycle_phases_ms": cyc,
               "profiled_solve_ms": e0.elapsed_time(e1),
               "model": {"sum_c_k": ph["f_leg"] + ph["g_leg"], "H_screen": 0.0, "H_check": ph["column_check"],
                         "H_compact": ph["plan"] + ph["emit_move"],
                         "note": "the row screen rides inside the f-leg: H_screen has no time of its own"}}
        # c_k as a function of the width A_k: mean update time of the cycles run at each width (binned by powers of two)
        widths = np.array(st["widths"][:len(trace)], dtype=np.int64)
        tr = np.array(trace[:len(widths)], dtype=np.float64)
        if len(widths):
            bins = {}
            for wd, ms_ in zip(widths, tr):
                key = 1 << int(np.ceil(np.log2(max(int(wd), 1))))
                bins.setdefault(key, []).append(ms_)
            out["c_k_by_width"] = [{"width_le": k, "cycles": len(v), "mean_update_us": 1e3 * float(np.mean(v))}
                                   for k, v in sorted(bins.items())]
        return out

    def parity(self, lanes=None, seconds=20.0):
        """The CUDA path against the oracle on this workload, inside a time bound: depths, potentials and the
        float64 residual of the emitted state, for as many lanes as the oracle finishes in `seconds`."""
        import oracle
        torch = self.torch
        w = self.w
        W, n, m, d = w.shape
        sb = self.batch("active")
        sb.drain()
        f, g = sb.potentials(f64=True); depth, status = sb.depths()
        sb.close()
        f, g, depth = f.cpu().numpy(), g.cpu().numpy(), depth.cpu().numpy()
        cores = os.cpu_count() or 1
        lanes = list(range(W)) if lanes is None else list(lanes)
        done, equal, off, worst_margin, pot, resid = 0, 0, 0, 0.0, 0.0, 0.0
        t0 = time.perf_counter()
        while done < len(lanes) and time.perf_counter() - t0 < seconds:
            sel = np.array(lanes[done:done + cores])
            r = oracle.solve_batch(w.x[sel], w.y[sel], w.a[sel], w.b[sel], w.eps[sel], w.tol, max_iter=w.max_iter)
            for i, t in enumerate(sel):
                if depth[t] == r.depth[i]:
                    equal += 1
                    num = max(np.abs(f[t] - r.f[i]).max(), np.abs(g[t] - r.g[i]).max())
                    den = max(np.abs(r.f[i]).max(), np.abs(r.g[i]).max(), float(w.eps[t]))
                    pot = max(pot, num / den)
                else:
                    off += 1
                    o = oracle.solve_lane(w.x[t], w.y[t], w.a[t], w.b[t], float(w.eps[t]), w.tol, max_iter=w.max_iter, history=True)
                    k = min(int(depth[t]), o.depth)
                    worst_margin = max(worst_margin, abs(max(o.hist_row[k - 1], o.hist_col[k - 1]) - w.tol) / w.tol)
                if n * m <= 1 << 20:
                    rr, rc = oracle.residuals(w.x[t], w.y[t], w.a[t], w.b[t], float(w.eps[t]), f[t], g[t])
                    resid = max(resid, max(rr, rc) / w.tol)
            done += len(sel)
        return {"against": "oracle, same inputs, this run", "lanes_compared": done, "of": W, "depths_equal": equal,
                "one_audit_away": off, "worst_margin_of_those": worst_margin, "max_potential_error": pot,
                "max_achieved_residual_over_tol": resid if resid > 0 else None, "seconds": time.perf_counter() - t0}

    def parity_stored(self):
        """Registration at full size: the oracle's stored results for a few lanes (tests/golden)."""
        path = os.path.join(ROOT, "tests", "golden", "registration_n8192.npz")
        if self.name != "registration" or not os.path.exists(path):
            return None
        z = np.load(path)
        w = self.w
        sb = self.batch("active")
        sb.drain()
        f, g = sb.potentials(f64=True); depth, _ = sb.depths()
        sb.close()
        f, g, depth = f.cpu().numpy(), g.cpu().numpy(), depth.cpu().numpy()
        equal, pot = 0, 0.0
        for i, t in enumerate(z["lanes"]):
            if int(depth[t]) == int(z["depth"][i]):
                equal += 1
                num = max(np.abs(f[t] - z["f"][i]).max(), np.abs(g[t] - z["g"][i]).max())
                den = max(np.abs(z["f"][i]).max(), np.abs(z["g"][i]).max(), float(w.eps[t]))
                pot = max(pot, num / den)
        return {"against": "oracle results stored by tests/golden/make_registration_golden.py (one lane is ~20 core-minutes)",
                "lanes_compared": int(len(z["lanes"])), "of": w.shape[0], "depths_equal": equal,
                "one_audit_away": int(len(z["lanes"])) - equal, "max_potential_error": pot}

    def cpu_baseline(self, seconds=10.0):
        """The oracle on the host cores, on a bounded sample of this workload."""
        import oracle
        w = self.w
        W, n, m, d = w.shape
        cores = os.cpu_count() or 1
        sel, cap, what = reference_sample(self.name, w, cores)
        done, units, threads = 0, 0.0, 1
        t0 = time.perf_counter()
        while done < len(sel) and time.perf_counter() - t0 < seconds:
            s = sel[done:done + cores]
            r = oracle.solve_batch(w.x[s], w.y[s], w.a[s], w.b[s], w.eps[s], w.tol, max_iter=cap)
            units += float(r.depth.sum()) * n * m
            threads = max(threads, r.threads)
            done += len(s)
        dt = time.perf_counter() - t0
        return {"value": units / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                "sample": f"{done} of {W} lanes, {what}"}


def e2e_host(R, args, flush, world, reps):
    """End to end through the host-buffer C call: pinned host inputs, copies inside the timed region."""
    torch, B, w, dev = R.torch, R.B, R.w, R.dev
    W, n, m, d = w.shape
    cfg = B.make_config(W, n, m, d, bf16=w.xy_dtype == "bf16", mode=args.mode, compute=args.compute,
                        max_iter=w.max_iter, stream=torch.cuda.current_stream().cuda_stream)
    need = B.sinkhorn_batch_host_workspace_bytes(cfg)
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    cfg.workspace, cfg.workspace_bytes = ws.data_ptr(), need
    pin = lambda v: torch.from_numpy(v).pin_memory()
    hx = (torch.from_numpy(w.x_bits.view(np.int16)) if w.xy_dtype == "bf16" else torch.from_numpy(w.x)).pin_memory()
    hy = (torch.from_numpy(w.y_bits.view(np.int16)) if w.xy_dtype == "bf16" else torch.from_numpy(w.y)).pin_memory()
    ha, hb, he = pin(w.a), pin(w.b), pin(w.eps)
    of = torch.empty(W, n, dtype=torch.float32).pin_memory(); og = torch.empty(W, m, dtype=torch.float32).pin_memory()
    od = torch.empty(W, dtype=torch.int32).pin_memory(); os_ = torch.empty(W, dtype=torch.int32).pin_memory()
    orr = torch.empty(W, dtype=torch.float32).pin_memory(); orc = torch.empty(W, dtype=torch.float32).pin_memory()
    p = lambda v: ctypes.c_void_p(v.data_ptr())
    slots = ctypes.c_longlong(0); cyc = ctypes.c_int(0)
    e2e_t = []
    for it in range(3 + reps):
        flush.fill_(1); torch.cuda.synchronize()
        t0 = time.perf_counter()
        rc = B.lib.sinkhorn_batch_solve_host(p(hx), p(hy), p(ha), p(hb), p(he), w.tol, ctypes.byref(cfg),
                                             p(of), p(og), p(od), p(os_), p(orr), p(orc),
                                             ctypes.byref(slots), ctypes.byref(cyc))
        dt = time.perf_counter() - t0
        if rc != 0:
            raise SystemExit("solve_host failed: " + B.lib.sinkhorn_batch_last_error(None).decode())
        if it >= 3:
            e2e_t.append(dt)
    e2e_ms = 1e3 * float(np.mean(e2e_t))
    h2d = hx.numel() * hx.element_size() + hy.numel() * hy.element_size() + 4 * (ha.numel() + hb.numel() + he.numel())
    d2h = 4 * (of.numel() + og.numel() + 4 * W)
    return {"value": world * slots.value * n * m / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "note": "host clock around sinkhorn_batch_solve_host, pinned buffers, rank 0"}


def tol_sweep_rows(R, reps, modes=("static", "masked", "masked_exit", "active")):
    """Completion-depth disagreement table: every tolerance of the grid in every mode."""
    from paper_2607_24741_b200 import workloads as wlmod
    torch = R.torch
    W = R.w.shape[0]
    rows = []
    for tol in wlmod.SWEEP_TOLS:
        row = {"tol": tol}
        for mode in modes:
            best, info = None, None
            for rep in range(reps):
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                sb = R.batch(mode, tol)
                sb.drain()
                e1.record(); torch.cuda.synchronize()
                ms_ = e0.elapsed_time(e1)
                best = ms_ if best is None or ms_ < best else best
                depth, status = sb.depths(); st = sb.stats()
                info = {"slots": st["slots"], "l_max": st["cycles"], "sum_depth": int(depth.sum().item()),
                        "done": int((status == 1).sum().item())}
                sb.close()
            row[mode] = {"ms": best, **info}
        row["W_lmax"] = W * row["active"]["l_max"]
        row["removed_slots"] = row["static"]["slots"] - row["active"]["slots"]
        row["static_over_active"] = row["static"]["ms"] / row["active"]["ms"]
        row["masked_over_active"] = row["masked"]["ms"] / row["active"]["ms"]
        if "masked_exit" in row:
            row["masked_exit_over_active"] = row["masked_exit"]["ms"] / row["active"]["ms"]
        rows.append(row)
    return rows


def workload_entry(name, args, dev, flush, unit_rates, local_rank, headline=None):
    """Everything the line reports about one of the five configurations."""
    R = headline["runner"] if headline else Runner(name, args, dev)
    w = R.w
    W, n, m, d = w.shape
    small = W * n * m < (1 << 27)
    steps = 9 if small else 3
    # Solves of a millisecond or two are timed while the clock sampler's nvidia-smi calls run beside
    # them, and one such call can hold a launch up for milliseconds: the entries of `workloads` other
    # than the headline therefore report the MEDIAN step (the mean is kept beside it).
    median = lambda v: float(sorted(v)[len(v) // 2])
    with ClockSampler(local_rank) as clk:
        if headline:
            ms, info = headline["ms"], headline["info"]
            ms_mean = ms
        else:
            ms_mean, info, _ = R.timed("active", steps, 3, flush)
            ms = median(R.last_step_ms)
        controls = {}
        for mode in ("static", "masked"):
            cmean, cinfo, _ = R.timed(mode, steps if small else 3, 3, flush)
            controls[mode] = {"ms": cmean if headline else median(R.last_step_ms), "ms_mean": cmean, "slots": cinfo["slots"]}
        roof, dtype, arith = R.roofline(unit_rates)
    entry = {"shape": {"W": W, "n": n, "m": m, "d": d, "tol": w.tol, "xy_dtype": w.xy_dtype}, "arithmetic": arith,
             "active": {"ms": ms, "ms_mean": ms_mean, "stat": "mean of steps" if headline else "median of steps",
                        "slots": info["slots"], "cycles": info["cycles"], "sum_depth": info["sum_depth"],
                        "lanes_done": info["done"], "create_ms": info["create_ms"],
                        "updates_per_s": info["slots"] * n * m / (ms * 1e-3)},
             "static": controls["static"], "masked": controls["masked"],
             "static_over_active": controls["static"]["ms"] / ms, "masked_over_active": controls["masked"]["ms"] / ms,
             "dominant_kernel": {"kernel": roof["kernel"], "ms_per_launch": roof["ms_per_launch"],
                                 "g_leg_ms_per_launch": roof["g_leg_ms_per_launch"],
                                 "frac_exp_roofline": roof["exp_frac"],
                                 "frac_binding": roof["frac"], "binding": roof.get("binding_unit", roof["bound"]),
                                 "frac_of_measured_unit_rates": roof.get("frac_of_measured_unit_rates")},
             "phases": R.phases("active"), "clocks": clk.summary()}
    # break-even condition of the time model (Eq. 12): the update time saved by running at the survivor
    # width A_k instead of W must exceed what screening, checking and compaction cost
    c_w = roof["ms_per_launch"] + roof["g_leg_ms_per_launch"]
    mdl = entry["phases"]["model"]
    saved = info["cycles"] * c_w - mdl["sum_c_k"]
    overhead = mdl["H_screen"] + mdl["H_check"] + mdl["H_compact"]
    entry["break_even"] = {"c_W_ms_per_cycle": c_w, "cycles": info["cycles"], "sum_k_c_W_minus_c_Ak_ms": saved,
                           "H_screen_plus_H_check_plus_H_compact_ms": overhead, "holds": bool(saved > overhead),
                           "note": "c_k(A_k) and the H terms from the profiled solve (one launch per leg, no overlap); "
                                   "c_k(W) = f-leg + g-leg at full width, timed alone"}
    if name == "registration":
        entry["parity"] = R.parity_stored()
    elif name == "feature":
        entry["parity"] = R.parity(lanes=range(0, W, 8), seconds=25.0)
    elif name == "sweep":
        entry["parity"] = R.parity(lanes=range(0, W, 16), seconds=25.0)
    else:
        entry["parity"] = R.parity(seconds=15.0)
    if name == "sweep":
        entry["tol_sweep"] = tol_sweep_rows(R, 1)
    return entry, roof, dtype


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=list(ALL))
    ap.add_argument("--mode", default=None, choices=["active", "masked", "static", "masked_exit"])
    ap.add_argument("--compute", default="auto", choices=["auto", "f32", "mixed", "f64", "tensor"])
    ap.add_argument("--only", action="store_true", help="measure --workload only (no `workloads` object)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tol", type=float, default=None, help="override the workload's stopping tolerance")
    ap.add_argument("--tol-sweep", action="store_true",
                    help="completion-depth disagreement report: every tolerance of the sweep grid in static, "
                         "masked and active mode, slots spent against W*l_max and sum l_t (one JSON line)")
    ap.add_argument("--width-sweep", action="store_true",
                    help="width report: W in {1,2,4,8,16} lanes of the registration law at n = 4096, solved "
                         "one lane at a time (width-one), static-packed and active-packed (one JSON line)")
    ap.add_argument("--audit-arms", action="store_true",
                    help="time the audit policies on --workload: fused row screen + column check of flagged lanes "
                         "(default) against a full two-sided check of every lane, each at every cycle and every 4th")
    ap.add_argument("--kernel-only", action="store_true",
                    help="only create the batch and time the update kernel (few launches; for profiler captures); "
                         "with --mode active: three 32-cycle launches of the multi-cycle kernel instead")
    ap.add_argument("--move-only", action="store_true",
                    help="a short ACTIVE solve of the first --lanes lanes with phase timing: emission/compaction "
                         "bytes, time and GB/s (few launches; for profiler captures of the compaction kernel)")
    ap.add_argument("--lanes", type=int, default=0, help="with --move-only / --kernel-only: use the first LANES lanes only")
    ap.add_argument("--unit-rates", action="store_true", help="only run the unit-rate self-test (one JSON line)")
    ap.add_argument("--refill", action="store_true",
                    help="stream all lanes of --workload through a batch of a quarter as many slots, new problems replacing "
                         "finished lanes, against the same lanes as four batches one after the other and as one wide batch")
    ap.add_argument("--shadow-replay", action="store_true",
                    help="replay a solve of the first --lanes lanes (default 256) cycle by cycle and compare, at every audit, "
                         "the fused row screen with the row residual computed directly from the potentials")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.mode is None:
        args.mode = "static" if args.kernel_only else "active"   # --kernel-only times the per-leg kernel unless --mode active is given

    rank = int(os.environ.get("RANK", "0")); world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2607_24741_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    if args.unit_rates:
        ur = B.unit_rates(dev)
        f_hz = peaks()["sm_max_mhz"] * 1e6
        print(json.dumps({"report": "unit-rates", "ops_per_s": ur,
                          "lanes_per_clk_per_sm_at_max_clock": {k: v / (SM_COUNT * f_hz) for k, v in ur.items()},
                          "nominal_lanes_per_clk_per_sm": {"ffma": FP32_LANES, "ffma2": FP32_LANES, "dfma": FP64_LANES, "ex2": MUFU_LANES}}),
              flush=True)
        return
    if args.width_sweep:
        from paper_2607_24741_b200 import workloads as wlmod
        big = wlmod.make("registration", W=16, n=4096)
        tt = lambda v: torch.from_numpy(v).to(dev)
        X, Y, A_, B_, E_ = tt(big.x), tt(big.y), tt(big.a), tt(big.b), tt(big.eps)

        def run(sl, mode):
            best = None
            for rep in range(2):
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                sb = B.SinkhornBatch(X[sl], Y[sl], A_[sl], B_[sl], E_[sl], big.tol, mode=mode, compute=args.compute,
                                     max_iter=big.max_iter)
                sb.drain()
                e1.record(); torch.cuda.synchronize()
                ms_ = e0.elapsed_time(e1)
                st = sb.stats(); sb.close()
                best = ms_ if best is None or ms_ < best else best
            return best, st["slots"], st["cycles"]

        rows = []
        for Wd in (1, 2, 4, 8, 16):
            one = sum(run(slice(t0, t0 + 1), "active")[0] for t0 in range(Wd))
            st_ms, st_slots, lmax = run(slice(0, Wd), "static")
            ac_ms, ac_slots, _ = run(slice(0, Wd), "active")
            rows.append({"W": Wd, "width_one_ms": one, "static_ms": st_ms, "active_ms": ac_ms, "l_max": lmax,
                         "static_slots": st_slots, "active_slots": ac_slots,
                         "width_one_over_static": one / st_ms, "static_over_active": st_ms / ac_ms,
                         "width_one_over_active": one / ac_ms})
        print(json.dumps({"report": "width-sweep", "law": "registration", "n": 4096, "d": 3, "rows": rows}), flush=True)
        return

    R = Runner(args.workload, args, dev, tol=args.tol)
    w = R.w
    if args.shadow_replay and not args.lanes:
        args.lanes = min(256, w.shape[0])
    if args.lanes:
        L = args.lanes
        R.x, R.y, R.a, R.b, R.eps = R.x[:L].contiguous(), R.y[:L].contiguous(), R.a[:L].contiguous(), R.b[:L].contiguous(), R.eps[:L].contiguous()
        w.x, w.y, w.a, w.b, w.eps = w.x[:L], w.y[:L], w.a[:L], w.b[:L], w.eps[:L]
    W, n, m, d = w.shape
    if args.tol_sweep:
        print(json.dumps({"report": "tol-sweep", "workload": args.workload, "W": W, "n": n, "m": m, "d": d,
                          "rows": tol_sweep_rows(R, 3)}), flush=True)
        return
    if args.audit_arms:
        rows, ref_depth = [], {}
        for every in (1, 4):
            for arm, screen in (("screen", 0.0), ("full_check", 1e30)):
                best, info, depth = None, None, None
                for rep in range(3):
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    sb = R.batch(args.mode, audit_every=every, tol_screen=screen)
                    sb.drain()
                    e1.record(); torch.cuda.synchronize()
                    ms_ = e0.elapsed_time(e1)
                    best = ms_ if best is None or ms_ < best else best
                    depth, status = sb.depths(); st = sb.stats()
                    info = {"slots": st["slots"], "cycles": st["cycles"], "pair_terms": st["pair_terms"],
                            "done": int((status == 1).sum().item())}
                    sb.close()
                ref_depth.setdefault(every, depth)
                # pair terms beyond the two legs of every slot are the column checks
                check_terms = info["pair_terms"] - 2 * info["slots"] * n * m
                rows.append({"audit_every": every, "arm": arm, "ms": best, **info, "column_check_pair_terms": check_terms,
                             "depths_equal_to_screen_arm": bool((depth == ref_depth[every]).all().item())})
        print(json.dumps({"report": "audit-arms", "workload": args.workload, "mode": args.mode, "W": W, "n": n, "m": m,
                          "d": d, "tol": w.tol, "rows": rows}), flush=True)
        return
    if args.shadow_replay:
        print(json.dumps(shadow_replay(R, args)), flush=True)
        return
    if args.refill:
        print(json.dumps(refill_report(R, args)), flush=True)
        return
    if args.kernel_only and args.mode == "active":
        # a few multi-cycle launches of the ACTIVE path (for profiler captures of the cluster kernels)
        sb = R.batch("active")
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sb.step(32); torch.cuda.synchronize()
        e0.record(); sb.step(32); sb.step(32); e1.record(); torch.cuda.synchronize()
        out = {"workload": args.workload, "arithmetic": sb.arithmetic(), "cycles": 64,
               "us_per_cycle": 1e3 * e0.elapsed_time(e1) / 64, "lanes_left": sb.active()}
        sb.close()
        print(json.dumps(out), flush=True)
        return
    if args.kernel_only:
        sb = R.batch("static")
        sb.step(2)
        out = {"workload": args.workload, "arithmetic": sb.arithmetic(),
               "f_leg_ms": sb.profile_update(leg=0, reps=3), "g_leg_ms": sb.profile_update(leg=1, reps=3)}
        sb.close()
        print(json.dumps(out), flush=True)
        return
    if args.move_only:
        ph = R.phases("active")
        sb = R.batch("active"); sb.drain(); st = sb.stats(widths_cap=200000); depth, _ = sb.depths(); sb.close()
        moves = move_accounting(w, st["widths"], depth.cpu().numpy(), R)
        ms = ph["ms"]["emit_move"]
        out = {"report": "emit-move", "workload": args.workload, "W": W, "n": n, "m": m, "d": d, **moves,
               "emit_move_ms_total": ms, "plan_ms_total": ph["ms"]["plan"],
               "GB_per_s_over_launches_that_moved": (moves["bytes_moved_total"] + moves["bytes_emitted_total"]) / 1e9 / (ms * 1e-3) if ms > 0 else None,
               "hbm_peak_GB_per_s": peaks()["hbm_gbs"], "phases": ph}
        print(json.dumps(out), flush=True)
        return

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > 126 MB L2
    with ClockSampler(local_rank) as clk:
        ms, info, launches = R.timed(args.mode, args.steps, args.warmup, flush, dist if world > 1 else None)
    clocks = clk.summary()
    units = float(info["slots"]) * n * m
    ms_all, units_all = aggregate(dist if world > 1 else None, ms, units)
    value = units_all / (ms_all * 1e-3)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_all, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",   # dtype refined below from the batch
            "config": {"workload": args.workload, "W": W, "n": n, "m": m, "d": d, "tol": w.tol,
                       "mode": args.mode, "compute": args.compute, "xy_dtype": w.xy_dtype,
                       "slots": info["slots"], "cycles": info["cycles"], "sum_depth": info["sum_depth"],
                       "lanes_done": info["done"], "l2": "256 MB buffer written between steps",
                       "parallelism": f"replicas x{world}"},
            "clocks": clocks, "gpu_launches": launches}

    if rank == 0:
        line["e2e"] = e2e_host(R, args, flush, world, max(3, min(args.steps // 2, 6)))
        unit_rates = B.unit_rates(dev)
        f_hz = peaks()["sm_max_mhz"] * 1e6
        line["unit_rates"] = {"lanes_per_clk_per_sm_at_max_clock": {k: round(v / (SM_COUNT * f_hz), 2) for k, v in unit_rates.items()},
                              "nominal": {"ffma": FP32_LANES, "ffma2": FP32_LANES, "dfma": FP64_LANES, "ex2": MUFU_LANES},
                              "how": "register-only loops of one instruction kind, event-timed (library self-test)"}
        if args.only or world > 1 or args.mode != "active":
            roof, dtype, _ = R.roofline(unit_rates)
            line["roofline"], line["dtype"] = roof, dtype
            ctl = {}
            for mode in ("static", "masked"):
                cms, cinfo, _ = R.timed(mode, 3, 3, flush)
                ctl[mode] = {"ms": cms, "slots": cinfo["slots"]}
            ctl[args.mode] = {"ms": ms, "slots": info["slots"]}
            line["controls"] = ctl
            line["phases"] = R.phases(args.mode if args.mode != "masked_exit" else "masked")
        else:
            entries = {}
            for name in ALL:
                head = {"runner": R, "ms": ms, "info": info} if name == args.workload else None
                entry, roof, dtype = workload_entry(name, args, dev, flush, unit_rates, local_rank, head)
                entries[name] = entry
                if name == args.workload:
                    line["roofline"], line["dtype"] = roof, dtype
                    line["controls"] = {"static": entry["static"], "masked": entry["masked"],
                                        "active": {"ms": ms, "slots": info["slots"]}}
                    line["phases"] = entry["phases"]
                    line["parity"] = entry["parity"]
                torch.cuda.empty_cache()
            line["workloads"] = entries
        # ---- the oracle on the host cores, bounded sample
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = R.cpu_baseline(10.0)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def shadow_replay(R, args, max_cycles=4000):
    """Shadow replay of the audit (the paper's attribution campaign counts screen-negative audits that a
    full check would already have released, and the largest gap between the screen and the full row
    residual).  Lanes stay in place (MASKED), one cycle per step; after every cycle the row residual of the
    current state is computed DIRECTLY from its potentials (a float64 pass over all pairs,
    sinkhorn_row_residual_static), and one cycle later the library reports what its fused screen made of
    that same state."""
    torch, B, w = R.torch, R.B, R.w
    W, n, m, d = w.shape
    if W > 256 or n > 8192:
        raise SystemExit("--shadow-replay: at most 256 lanes (use --lanes) of at most 8192 points")
    x32, y32 = R.x.float(), R.y.float()
    sb = R.batch("masked")
    tol = w.tol
    negatives = missed_ready = early_ready = events = 0
    worst, worst_rel = 0.0, 0.0
    direct_prev = None
    running = torch.ones(W, dtype=torch.bool, device=R.dev)
    for k in range(1, max_cycles + 1):
        sb.step(1)
        if direct_prev is not None:
            screen, _, _ = sb.last_audit()                   # the screen of the state after k-1 cycles
            sel = running & ~torch.isnan(screen)
            dp, sc = direct_prev[sel].double(), screen[sel].double()
            events += int(sel.sum().item())
            neg = sc > tol
            negatives += int(neg.sum().item())
            missed_ready += int((neg & (dp <= tol)).sum().item())
            early_ready += int((~neg & (dp > tol)).sum().item())
            if dp.numel():
                gap = (sc - dp).abs()
                worst = max(worst, float(gap.max().item()))
                worst_rel = max(worst_rel, float((gap / dp.clamp_min(1e-300)).max().item()))
        depth, status = sb.depths()
        running = status == 0
        if not bool(running.any().item()):
            break
        f, g = sb.potentials(f64=True)
        direct_prev = B.sinkhorn_row_residual_static(x32, y32, R.a, f, g, R.eps)
    cycles = sb.stats()["cycles"]
    arith = sb.arithmetic()
    sb.close()
    return {"report": "shadow-replay", "workload": args.workload, "W": W, "n": n, "m": m, "d": d, "tol": tol,
            "arithmetic": arith, "cycles": cycles, "lane_audits_compared": events, "screen_negative": negatives,
            "missed_ready": missed_ready, "screen_positive_but_direct_above_tol": early_ready,
            "max_abs_screen_minus_direct": worst, "max_rel_screen_minus_direct": worst_rel,
            "paper_in_kind": {"screen_negative": 1488, "missed_ready": 0, "max_discrepancy": 1.86e-7}}


def refill_report(R, args):
    """All W lanes of the workload through S = W/4 slots, three ways: one wide batch (W slots), four batches
    of S lanes one after the other, and one batch of S slots whose finished lanes are replaced by the next
    problems whenever at least S/8 slots are free (checked every 16 cycles)."""
    torch, B, w = R.torch, R.B, R.w
    W, n, m, d = w.shape
    S = max(1, W // 4)
    x, y, a, b, eps = R.x, R.y, R.a, R.b, R.eps

    def timed(fn):
        best, out = None, None
        for rep in range(2):
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); out = fn(); e1.record(); torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            best = ms if best is None or ms < best else best
        return best, out

    def wide():
        sb = R.batch("active"); sb.drain(); st = sb.stats(); d_, _ = sb.depths(); sb.close()
        return st["slots"], st["cycles"], d_

    def quarters():
        slots = cyc = 0
        for q in range(0, W, S):
            sl = slice(q, min(W, q + S))
            sb = B.SinkhornBatch(x[sl], y[sl], a[sl], b[sl], eps[sl], w.tol, compute=args.compute, max_iter=w.max_iter)
            sb.drain(); st = sb.stats(); sb.close()
            slots += st["slots"]; cyc += st["cycles"]
        return slots, cyc, None

    def refilled():
        sb = B.SinkhornBatch(x[:S], y[:S], a[:S], b[:S], eps[:S], w.tol, compute=args.compute, max_iter=w.max_iter,
                             lane_capacity=W)
        nxt, refills = S, 0
        while nxt < W:
            sb.step(16)
            free = S - sb.active()
            if free >= max(1, S // 8) or free == S:
                c = min(free, W - nxt)
                sl = slice(nxt, nxt + c)
                sb.refill(x[sl], y[sl], a[sl], b[sl], eps[sl]); nxt += c; refills += 1
        sb.drain(); st = sb.stats(); d_, _ = sb.depths(); sb.close()
        return st["slots"], st["cycles"], d_, refills

    ms_w, (sl_w, cy_w, dw) = timed(wide)
    ms_q, (sl_q, cy_q, _) = timed(quarters)
    ms_r, (sl_r, cy_r, dr, refills) = timed(refilled)
    return {"report": "refill", "workload": args.workload, "W": W, "slots_held": S, "n": n, "m": m, "d": d,
            "one_wide_batch": {"ms": ms_w, "slots": sl_w, "cycles": cy_w},
            "four_batches_in_turn": {"ms": ms_q, "slots": sl_q, "cycles": cy_q},
            "refilled_batch": {"ms": ms_r, "slots": sl_r, "cycles": cy_r, "refills": refills,
                               "depths_equal_to_wide_batch": bool((dw == dr).all().item())},
            "in_turn_over_refilled": ms_q / ms_r, "refilled_over_wide": ms_r / ms_w}


def move_accounting(w, widths, depth, R):
    """Bytes the retirements of an ACTIVE solve emit and move: a retiree's potentials are written out
    (8 (n + m) bytes); a retiree whose slot lies below the new width is refilled by one survivor's
    whole state (read + write)."""
    W, n, m, d = w.shape
    sb = R.batch("active")
    arith = sb.arithmetic()
    sb.close()
    ts = 8 if arith in ("mixed", "f64") else 4
    np_, mp_ = (n + 3) // 4 * 4, (m + 3) // 4 * 4
    if arith == "tensor":
        coords = ((n + 127) // 128 + (m + 127) // 128) * d * 256
    else:
        DP = next(o for o in (2, 3, 4, 8, 16, 32, 1 << 30) if d <= o)
        DP = DP if d <= 32 else (d + 15) // 16 * 16
        coords = DP * (np_ + mp_) * ts
    lane_bytes = coords + (np_ + mp_) * (3 * 8) + np_ * (8 + 2 * ts) + mp_ * (8 + 2 * ts)
    depth = np.sort(np.asarray(depth))
    retire_events = len(np.unique(depth))
    # an upper bound on the moves: one per retiree that is not among the last slots; the exact count depends on slot order
    return {"arithmetic": arith, "lane_state_bytes": int(lane_bytes), "retirements": int(len(depth)),
            "audits_with_a_retirement": int(retire_events),
            "bytes_emitted_total": int(len(depth) * 8 * (n + m)),
            "bytes_moved_total": int(2 * lane_bytes * max(0, len(depth) - 1)),
            "note": "moves counted as one per retirement (upper bound: a retiree in the last slots needs none)"}


if __name__ == "__main__":
    main()
