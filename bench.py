#!/usr/bin/env python
"""Benchmark of the batched shrinking-active-set Sinkhorn hot path on B200.

One "step" = one whole solve of one synthetic batch: create (layout kernels), every cycle
of update / screen / two-sided check / retirement / compaction until all lanes have passed,
results written.  Metric: lane*n*m updates per second, counting one unit per executed
lane-cycle (slot) and point pair, i.e. (sum_k A_k) * n * m / time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload sensor] [--mode active]
  python bench.py --impl reference ...     # the float64 CPU oracle on the same workload

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

# DRAM bytes (read + write) of ONE full-width f-leg launch of the dominant kernel, taken from ncu
# captures of `bench.py --workload <name> --kernel-only` (one launch each; they equal the lanes'
# operands read once)
NCU_TRAFFIC_BYTES = {"sensor": 20.5e6, "registration": 13.7e6, "sweep": 42.0e6, "feature": 193.3e6}

# nominal unit counts (148 SMs, 128 FP32 lanes and 16 special-function lanes per SM per clock,
# 64 FP64 lanes) at the maximum SM clock; the fraction reported is against these
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


def run_reference(args, rank, world):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of lanes."""
    if rank != 0:
        return
    import oracle
    w = make_workload(args.workload)
    W, n, m, d = w.shape
    cores = os.cpu_count() or 1
    per_lane = 3.0 * n * m * 12e-9 * 400 + n * m * d * 2e-9       # crude cost guess, only to bound the sample
    lanes = int(max(1, min(W, cores * max(1, int(4.0 / max(per_lane, 1e-3))))))
    if args.workload == "sensor":
        lanes = min(W, max(cores, 64))
    sel = np.arange(lanes)
    times, units = [], 0
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        r = oracle.solve_batch(w.x[sel], w.y[sel], w.a[sel], w.b[sel], w.eps[sel], w.tol, max_iter=w.max_iter)
        dt = time.perf_counter() - t0
        if it >= args.warmup:
            times.append(dt)
            units = int(r.depth.sum()) * n * m
    ms = 1e3 * sum(times) / len(times)
    val = units / (ms * 1e-3)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "W": W, "n": n, "m": m, "d": d, "tol": w.tol,
                       "sample": f"lanes 0..{lanes - 1} of {W}"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": r.threads, "kind": "oracle",
                             "sample": f"lanes 0..{lanes - 1} of {W}, every lane run to its own depth"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="sensor", choices=["tiny", "sensor", "feature", "registration", "sweep"])
    ap.add_argument("--mode", default="active", choices=["active", "masked", "static", "masked_exit"])
    ap.add_argument("--compute", default="auto", choices=["auto", "f32", "mixed", "f64", "tensor"])
    ap.add_argument("--no-controls", action="store_true", help="skip the static / masked control timings")
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
                    help="only create the batch and time the update kernel (few launches; for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

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
    w = make_workload(args.workload)
    if args.tol is not None:
        w.tol = args.tol
    W, n, m, d = w.shape
    t = lambda v: torch.from_numpy(v).to(dev)
    x, y = t(w.x), t(w.y)
    if w.xy_dtype == "bf16":
        x, y = x.bfloat16(), y.bfloat16()
    a, b, eps = t(w.a), t(w.b), t(w.eps)
    if args.tol_sweep:
        from paper_2607_24741_b200 import workloads as wlmod
        rows = []
        for tol in wlmod.SWEEP_TOLS:
            row = {"tol": tol}
            for mode in ("static", "masked", "masked_exit", "active"):
                best, info = None, None
                for rep in range(3):
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    sb = B.SinkhornBatch(x, y, a, b, eps, tol, mode=mode, compute=args.compute, max_iter=w.max_iter)
                    sb.drain()
                    e1.record(); torch.cuda.synchronize()
                    ms_ = e0.elapsed_time(e1)
                    if best is None or ms_ < best:
                        best = ms_
                    depth, status = sb.depths(); st = sb.stats()
                    info = {"slots": st["slots"], "l_max": st["cycles"], "sum_depth": int(depth.sum().item()),
                            "done": int((status == 1).sum().item())}
                    sb.close()
                row[mode] = {"ms": best, **info}
            row["W_lmax"] = W * row["active"]["l_max"]
            row["removed_slots"] = row["static"]["slots"] - row["active"]["slots"]
            row["static_over_active"] = row["static"]["ms"] / row["active"]["ms"]
            row["masked_over_active"] = row["masked"]["ms"] / row["active"]["ms"]
            row["masked_exit_over_active"] = row["masked_exit"]["ms"] / row["active"]["ms"]
            rows.append(row)
        print(json.dumps({"report": "tol-sweep", "workload": args.workload, "W": W, "n": n, "m": m, "d": d,
                          "rows": rows}), flush=True)
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
                    sb = B.SinkhornBatch(x, y, a, b, eps, w.tol, mode=args.mode, compute=args.compute, max_iter=w.max_iter,
                                         audit_every=every, tol_screen=screen)
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
    if args.kernel_only:
        sb = B.SinkhornBatch(x, y, a, b, eps, w.tol, mode="static", compute=args.compute, max_iter=w.max_iter)
        sb.step(2)
        out = {"workload": args.workload, "arithmetic": sb.arithmetic(),
               "f_leg_ms": sb.profile_update(leg=0, reps=3), "g_leg_ms": sb.profile_update(leg=1, reps=3)}
        sb.close()
        print(json.dumps(out), flush=True)
        return
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > 126 MB L2

    def solve(mode, collect=False):
        sb = B.SinkhornBatch(x, y, a, b, eps, w.tol, mode=mode, compute=args.compute, max_iter=w.max_iter)
        sb.drain()
        out = None
        if collect:
            st = sb.stats()
            depth, status = sb.depths()
            out = {"slots": st["slots"], "cycles": st["cycles"], "pair_terms": st["pair_terms"],
                   "launches": sb.launch_count(), "sum_depth": int(depth.sum().item()),
                   "done": int((status == 1).sum().item())}
        sb.close()
        return out

    def timed(mode, steps, warmup):
        info = None
        for _ in range(warmup):
            info = solve(mode, collect=True)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        total = 0.0
        launches = 0
        for _ in range(steps):
            flush.fill_(1)                                             # evict L2 between steps
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            solve(mode)
            e1.record()
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1)
            launches += info["launches"]
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        return total / steps, info, launches

    with ClockSampler(local_rank) as clk:
        ms, info, launches = timed(args.mode, args.steps, args.warmup)
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
        # ---- end to end through the host-buffer C call (pinned host memory, copies inside)
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
        for it in range(3 + max(3, args.steps // 2)):
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
        line["e2e"] = {"value": world * slots.value * n * m / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "note": "host clock around sinkhorn_batch_solve_host, pinned buffers, rank 0"}

        # ---- roofline of the dominant kernel (update kernel, f-leg at full width)
        sb = B.SinkhornBatch(x, y, a, b, eps, w.tol, mode="static", compute=args.compute, max_iter=w.max_iter)
        sb.step(2)
        k_ms = sb.profile_update(leg=0, reps=20)
        arith = sb.arithmetic()
        sb.close()
        pk = peaks()
        f_hz = pk["sm_max_mhz"] * 1e6
        pairs = float(W) * n * m
        # algorithmic work per pair: d FMAs for the cross term, then max, subtract, exponential, add
        # (float64 exponents: d FMAs + max + subtract on the half-rate FP64 pipe)
        wide = arith != "f32"
        inst_per_pair = d + 2 if wide else d + 3
        lanes = FP64_LANES if wide else FP32_LANES
        fp32_peak = SM_COUNT * lanes * f_hz
        mufu_peak = SM_COUNT * MUFU_LANES * f_hz
        achieved_inst = pairs * inst_per_pair / (k_ms * 1e-3)
        achieved_exp = pairs / (k_ms * 1e-3)
        bound_fp32 = inst_per_pair / lanes > 1.0 / MUFU_LANES
        line["dtype"] = {"f32": "f32", "mixed": "f64 exponents / f32 exp", "f64": "f64",
                         "tensor": "bf16 (f32 accumulate, f32 exp)"}[arith]
        if arith == "tensor":
            # the cross term is a dense bf16 contraction: 2*d flops per pair against the measured
            # cuBLAS bf16 burst throughput (kernel timed alone)
            tf = 2.0 * d * pairs / (k_ms * 1e-3) / 1e12
            line["roofline"] = {"bound": "tensor", "kernel": "update_tc_pair_kernel (f-leg, full width)",
                                "arithmetic": arith, "achieved": tf, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                                "frac": tf / pk["bf16_tflops"], "exp_frac": achieved_exp / mufu_peak,
                                "ms_per_launch": k_ms, "pairs_per_launch": pairs,
                                "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                                "peak_source": pk["source"] + " cuBLAS bf16 burst (MEASURED_PEAKS.json)"}
        else:
          line["roofline"] = {
            "bound": "alu", "kernel": "update_kernel (f-leg, full width)",
            "arithmetic": arith,
            "binding_unit": ("fp64 pipe" if wide else "fp32 pipe") if bound_fp32 else "special-function unit (ex2)",
            "achieved": (achieved_inst if bound_fp32 else achieved_exp) / 1e12,
            "peak": (fp32_peak if bound_fp32 else mufu_peak) / 1e12,
            "unit": "T lane-instr/s" if bound_fp32 else "T exp/s",
            "frac": (achieved_inst / fp32_peak) if bound_fp32 else (achieved_exp / mufu_peak),
            "exp_frac": achieved_exp / mufu_peak, "pipe_frac": achieved_inst / fp32_peak,
            "ms_per_launch": k_ms, "pairs_per_launch": pairs, "peak_clock_mhz": pk["sm_max_mhz"],
            "traffic": NCU_TRAFFIC_BYTES.get(args.workload), "traffic_unit": "bytes per launch (ncu)",
            "peak_source": "unit counts x max SM clock"}

        # ---- static / masked controls on the same kernels
        if not args.no_controls:
            ctl = {}
            for mode in ("static", "masked", "active"):
                cms, cinfo, _ = (ms, info, 0) if mode == args.mode else timed(mode, max(3, args.steps // 4), 3)
                ctl[mode] = {"ms": cms, "slots": cinfo["slots"]}
            line["controls"] = ctl

        # ---- the oracle on the host cores, bounded sample (about 10 s of wall time at most)
        if not args.no_cpu_baseline:
            import oracle
            cores = os.cpu_count() or 1
            cap = min(w.max_iter, 40) if n * m > 2048 * 2048 else w.max_iter
            done_lanes, units, threads = 0, 0.0, 1
            t0 = time.perf_counter()
            while done_lanes < W and time.perf_counter() - t0 < 8.0:
                sl = slice(done_lanes, min(W, done_lanes + cores))
                r = oracle.solve_batch(w.x[sl], w.y[sl], w.a[sl], w.b[sl], w.eps[sl], w.tol, max_iter=cap)
                units += float(r.depth.sum()) * n * m
                threads = max(threads, r.threads)
                done_lanes = sl.stop
            dt = time.perf_counter() - t0
            line["cpu_baseline"] = {"value": units / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                                    "sample": f"lanes 0..{done_lanes - 1} of {W}, each to its own depth"
                                              + (f" (capped at {cap} cycles)" if cap < w.max_iter else "")}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
