"""Shared helpers for the GPU parity tests: run a workload through the C-ABI binding and
through the CPU oracle on the same arrays, and compare the way the acceptance bar says.

Every comparison adds one entry to LEDGER: how many lanes were compared, how many stopped one
audit away from the oracle (each with the oracle's margin at the disputed audit), the largest
potential error and the largest residual deviations.  tests/test_yy_parity_ledger.py bounds
the totals and writes the table out, so that no near-threshold lane goes unreported."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

LEDGER: list[dict] = []

# The band inside which the acceptance bar itself allows a lane to stop one audit away.
ACCEPTANCE_BAND = 1e-6

# |r_col reported by the GPU - float64 column residual of the potentials it emitted|.  After a
# g-leg the column marginal is current (Eq. 4), so both are pure arithmetic error: the column
# check repeats the g-leg's sums in the GPU's arithmetic and finds (almost) nothing, while the
# float64 evaluation sees the g-leg's own error: 2^-22 per fp32 exponential, plus half an ulp of
# the scaled cost (up to 512, i.e. 2^-15 in the exponent) when the exponents are fp32 too.
# Float64: one ulp of an exponent of size C/eps (up to ~5e3 for eps = 0.01 at d = 40: 9e-13) in every
# plan entry, i.e. ~1e-12 in the column sums; ten times that is allowed.
RCOL_ABS = {"f64": 1e-11, "mixed": 5e-7, "f32": 1e-5, "tensor": 3e-5}     # observed: 1.6e-12, 8.9e-8, 1.9e-6, 1.1e-5

# Allowance on "float64 residual of the emitted state <= tol" (as a fraction of tol): the GPU stops a
# lane when ITS evaluation of the residual passes, so the float64 value may exceed tol by the
# evaluation error.  fp32 / mixed: observed up to 2e-5 of tol on the workloads, 5e-3 allowed.  Tensor
# cores: the fp32 accumulation of the 32 k-steps of a d = 512 dot product is the least accurate link
# (measured on the same inputs: the float64 column residual of an emitted state is 1.0e-5 on every
# lane, against 6.7e-7 with fp32 FMAs in the SIMT kernel), and the fused screen is off by up to
# 0.8 % of tol either way, so 1e-2 is allowed there.  The paper's answer to exactly this (Section 5:
# raw low-precision decisions flip near the threshold; a guard removes them) is the guard arm, which
# a test runs with NO allowance.
RESIDUAL_ALLOW = {"f64": 1e-9, "mixed": 5e-3, "f32": 5e-3, "tensor": 1e-2}


def run_gpu(w, mode="active", compute="auto", column_split=0, audit_every=1, tol_screen=0.0,
            max_iter=None, tol=None, widths_cap=200000, cost_form=0, warm=None, audit_initial=False,
            guard_band=0.0):
    import torch
    from paper_2607_24741_b200 import binding as B
    dev = torch.device("cuda:0")
    x = torch.from_numpy(w.x).to(dev); y = torch.from_numpy(w.y).to(dev)
    if w.xy_dtype == "bf16":
        x = x.bfloat16(); y = y.bfloat16()           # exact: values are bf16-representable
    a = torch.from_numpy(w.a).to(dev); b = torch.from_numpy(w.b).to(dev)
    eps = torch.from_numpy(w.eps).to(dev)
    sb = B.SinkhornBatch(x, y, a, b, eps, w.tol if tol is None else tol, mode=mode, compute=compute,
                         max_iter=w.max_iter if max_iter is None else max_iter,
                         audit_every=audit_every, tol_screen=tol_screen, column_split=column_split,
                         cost_form=cost_form, guard_band=guard_band)
    try:
        if warm is not None:
            sb.warm_start(torch.from_numpy(warm[0]).to(dev), torch.from_numpy(warm[1]).to(dev),
                          audit_initial=audit_initial)
        cycles = sb.drain()
        f, g = sb.potentials(f64=True)
        f32, g32 = sb.potentials()
        depth, status = sb.depths()
        rr, rc = sb.residuals()
        stats = sb.stats(widths_cap=widths_cap)
        left = sb.active()
        arith = sb.arithmetic()
        bad_strip = sb.check_guards()
    finally:
        sb.close()
    # no kernel of the solve wrote past the end of an array of the workspace (checked in every GPU run)
    assert bad_strip == -1, f"guard strip {bad_strip} of the workspace was overwritten"
    return dict(f=f.cpu().numpy(), g=g.cpu().numpy(), f32=f32.cpu().numpy(), g32=g32.cpu().numpy(),
                depth=depth.cpu().numpy(), status=status.cpu().numpy(), r_row=rr.cpu().numpy(),
                r_col=rc.cpu().numpy(), stats=stats, cycles=cycles, left=left, arith=arith)


def pot_err(f, g, fo, go, eps):
    """max(|df|_inf, |dg|_inf) / max(|f|_inf, |g|_inf, eps), per lane."""
    num = np.maximum(np.abs(f - fo).max(1), np.abs(g - go).max(1))
    den = np.maximum(np.maximum(np.abs(fo).max(1), np.abs(go).max(1)), eps)
    return num / den


def oracle_lanes(oracle, w, lanes, tol=None, max_iter=None, audit_every=1, tol_screen=0.0, warm=None,
                 audit_initial=False):
    """Per-lane oracle results with the neighbouring states (depth-1, depth, depth+1); lanes are
    independent problems (Eq. 2), so they are spread over the host cores, one whole lane each."""
    lanes = list(lanes)

    def one(t):
        kw = {}
        if warm is not None:
            kw = dict(f0=warm[0][t], g0=warm[1][t], audit_initial=audit_initial)
        return oracle.solve_lane(w.x[t], w.y[t], w.a[t], w.b[t], float(w.eps[t]),
                                 w.tol if tol is None else tol,
                                 max_iter=w.max_iter if max_iter is None else max_iter,
                                 audit_every=audit_every, tol_screen=tol_screen,
                                 neighbours=True, history=True, **kw)
    with ThreadPoolExecutor(max_workers=min(len(lanes), os.cpu_count() or 1) or 1) as ex:
        return dict(zip(lanes, ex.map(one, lanes)))


def miss_allowed(margin, decay, floor):
    """A lane may sit one audit away if the oracle's margin at the disputed audit is below the
    arithmetic's residual error: a floor, or for slowly converging lanes the fp32 exponential
    error 2^-22 accumulated over the ~1/decay cycles the iteration remembers (factor 4 slack)."""
    return margin <= max(floor, 4.0 * 2.0 ** -22 / max(decay, 1e-12))


def compare_lane(oracle, w, r, t, o, *, pot_tol, exact_depth, tol, audit_every=1, report_tol=None, entry=None):
    """One lane of the acceptance bar against an oracle result `o` (anything with depth, status, f, g,
    f_prev, g_prev, f_next, g_next and the history of max(r_row, r_col) in `hist`; an optional
    `stride` says that its potentials hold every stride-th point only).  Returns the miss record of a
    lane that stopped one audit away, else None."""
    st = int(getattr(o, "stride", 1))
    dg = int(r["depth"][t]); do = int(o.depth)
    assert r["status"][t] == o.status, (t, r["status"][t], o.status)
    miss = None
    if dg == do:
        fo, go = o.f, o.g
    else:
        assert not exact_depth, f"lane {t}: depth {dg} != oracle {do}"
        assert abs(dg - do) == audit_every, f"lane {t}: depth {dg} vs oracle {do}"
        fo, go = (o.f_prev, o.g_prev) if dg < do else (o.f_next, o.g_next)
        if audit_every == 1:
            hist = o.hist
            k = min(dg, do)                       # the audit the two sides disagree on
            margin = abs(hist[k - 1] - tol) / tol
            # relative decay of the oracle residual per cycle around that audit: an error injected
            # every cycle is remembered for about 1/decay cycles
            decay = abs(hist[max(k - 2, 0)] - hist[k - 1]) / tol if k >= 2 else 1.0
            miss = (t, dg, do, float(margin), float(decay))
    e = None
    if dg == do or audit_every == 1:
        e = pot_err(r["f"][t][None, ::st], r["g"][t][None, ::st], np.asarray(fo, np.float64)[None],
                    np.asarray(go, np.float64)[None], float(w.eps[t]))[0]
        assert e <= pot_tol, f"lane {t}: potential error {e:.3e} > {pot_tol}"
    if o.status == oracle.DONE:
        # the achieved two-sided residual, evaluated in float64 from the emitted potentials
        rr, rc = oracle.residuals(w.x[t], w.y[t], w.a[t], w.b[t], float(w.eps[t]), r["f"][t], r["g"][t])
        if report_tol is not None:
            # guard arm: the solve ran with a stricter threshold, the reported tolerance holds with no slack
            assert max(rr, rc) <= report_tol, (t, rr, rc)
        else:
            assert max(rr, rc) <= tol * (1 + RESIDUAL_ALLOW[r["arith"]]), (t, rr, rc)
        assert r["r_row"][t] <= tol
        assert abs(r["r_row"][t] - rr) <= 2e-2 * tol
        # the column half of the two-sided check (Eq. 5) as the GPU measured it
        assert np.isfinite(r["r_col"][t]) and r["r_col"][t] >= 0.0
        assert abs(float(r["r_col"][t]) - rc) <= RCOL_ABS[r["arith"]], (t, float(r["r_col"][t]), rc)
        if entry is not None:
            entry["max_residual_over_tol"] = float(max(entry["max_residual_over_tol"], max(rr, rc) / (report_tol or tol)))
            entry["max_rrow_dev_over_tol"] = float(max(entry["max_rrow_dev_over_tol"], abs(float(r["r_row"][t]) - rr) / tol))
            entry["max_rcol_dev"] = float(max(entry["max_rcol_dev"], abs(float(r["r_col"][t]) - rc)))
    if entry is not None and e is not None:
        entry["max_pot_err"] = max(entry["max_pot_err"], float(e))
    return miss


def new_entry(label, w, r, lanes, tol, floor):
    return dict(label=label, workload=w.name, shape=[int(v) for v in w.shape], arith=r["arith"], tol=float(tol), lanes=len(lanes),
                equal=0, misses=[], floor=floor, max_pot_err=0.0, max_residual_over_tol=0.0,
                max_rrow_dev_over_tol=0.0, max_rcol_dev=0.0)


def close_entry(entry, misses, floor):
    for (t, dg, do, margin, decay) in misses:
        entry["misses"].append(dict(lane=int(t), gpu=dg, oracle=do, margin=margin, decay=decay,
                                    inside_1e6_band=bool(margin <= ACCEPTANCE_BAND)))
        if floor is not None:
            assert miss_allowed(margin, decay, floor), \
                f"{entry['label']} lane {t}: gpu {dg} oracle {do} margin {margin:.2e} decay {decay:.2e}"
    entry["equal"] = entry["lanes"] - len(misses)
    LEDGER.append(entry)


def check_against_oracle(oracle, w, r, lanes, *, pot_tol, exact_depth, tol=None, max_iter=None,
                         audit_every=1, tol_screen=0.0, floor=None, label="", report_tol=None, warm=None,
                         audit_initial=False):
    """Acceptance bar on the given lanes.  Depths must be equal; where exact_depth is False a
    lane may be off by one audit, and every such lane is returned with the oracle's margin
    |r - tol|/tol at the two candidate depths (and, when `floor` is given, held to miss_allowed).
    Potentials are compared at the GPU's own depth (the oracle also emits its neighbours)."""
    tol = w.tol if tol is None else tol
    lanes = list(lanes)
    ref = oracle_lanes(oracle, w, lanes, tol, max_iter, audit_every, tol_screen, warm, audit_initial)
    entry = new_entry(label, w, r, lanes, tol, floor)
    misses = []
    for t in lanes:
        o = ref[t]
        o.hist = np.maximum(o.hist_row, o.hist_col)
        m = compare_lane(oracle, w, r, t, o, pot_tol=pot_tol, exact_depth=exact_depth, tol=tol,
                         audit_every=audit_every, report_tol=report_tol, entry=entry)
        if m is not None:
            misses.append(m)
    close_entry(entry, misses, floor)
    return misses


def check_accounting(oracle, r, W, mode):
    """Eq. 6-8: slots, widths and depths must agree exactly."""
    depth = r["depth"].astype(np.int64)
    s = oracle.slot_counts(depth)
    lmax = int(depth.max())
    assert r["cycles"] == lmax == r["stats"]["cycles"]
    if mode == "active":
        assert r["stats"]["slots"] == s["S_active"] == depth.sum()
        np.testing.assert_array_equal(np.array(r["stats"]["widths"]), s["widths"])
    else:
        assert r["stats"]["slots"] == s["S_static"] == W * lmax
        assert all(wd == W for wd in r["stats"]["widths"])
    assert r["left"] == 0
