"""Shared helpers for the GPU parity tests: run a workload through the C-ABI binding and
through the CPU oracle on the same arrays, and compare the way the acceptance bar says."""
from __future__ import annotations

import numpy as np


def run_gpu(w, mode="active", compute="auto", column_split=0, audit_every=1, tol_screen=0.0,
            max_iter=None, tol=None, widths_cap=200000, cost_form=0):
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
                         cost_form=cost_form)
    try:
        cycles = sb.drain()
        f, g = sb.potentials(f64=True)
        f32, g32 = sb.potentials()
        depth, status = sb.depths()
        rr, rc = sb.residuals()
        stats = sb.stats(widths_cap=widths_cap)
        left = sb.active()
    finally:
        sb.close()
    return dict(f=f.cpu().numpy(), g=g.cpu().numpy(), f32=f32.cpu().numpy(), g32=g32.cpu().numpy(),
                depth=depth.cpu().numpy(), status=status.cpu().numpy(), r_row=rr.cpu().numpy(),
                r_col=rc.cpu().numpy(), stats=stats, cycles=cycles, left=left)


def pot_err(f, g, fo, go, eps):
    """max(|df|_inf, |dg|_inf) / max(|f|_inf, |g|_inf, eps), per lane."""
    num = np.maximum(np.abs(f - fo).max(1), np.abs(g - go).max(1))
    den = np.maximum(np.maximum(np.abs(fo).max(1), np.abs(go).max(1)), eps)
    return num / den


def oracle_lanes(oracle, w, lanes, tol=None, max_iter=None, audit_every=1, tol_screen=0.0):
    """Per-lane oracle results with the neighbouring states (depth-1, depth, depth+1)."""
    out = {}
    for t in lanes:
        out[t] = oracle.solve_lane(w.x[t], w.y[t], w.a[t], w.b[t], float(w.eps[t]),
                                   w.tol if tol is None else tol,
                                   max_iter=w.max_iter if max_iter is None else max_iter,
                                   audit_every=audit_every, tol_screen=tol_screen,
                                   neighbours=True, history=True)
    return out


def check_against_oracle(oracle, w, r, lanes, *, pot_tol, exact_depth, tol=None, max_iter=None,
                         audit_every=1, tol_screen=0.0):
    """Acceptance bar on the given lanes.  Depths must be equal; where exact_depth is False a
    lane may be off by one audit, and every such lane is returned with the oracle's margin
    |r - tol|/tol at the two candidate depths so that the caller can bound and report it.
    Potentials are compared at the GPU's own depth (the oracle also emits its neighbours)."""
    tol = w.tol if tol is None else tol
    ref = oracle_lanes(oracle, w, lanes, tol, max_iter, audit_every, tol_screen)
    misses = []
    for t in lanes:
        o = ref[t]
        dg = int(r["depth"][t]); do = o.depth
        assert r["status"][t] == o.status, (t, r["status"][t], o.status)
        if dg == do:
            fo, go = o.f, o.g
        else:
            assert not exact_depth, f"lane {t}: depth {dg} != oracle {do}"
            assert abs(dg - do) == audit_every, f"lane {t}: depth {dg} vs oracle {do}"
            fo, go = (o.f_prev, o.g_prev) if dg < do else (o.f_next, o.g_next)
            if audit_every == 1:
                hist = np.maximum(o.hist_row, o.hist_col)
                k = min(dg, do)                       # the audit the two sides disagree on
                margin = abs(hist[k - 1] - tol) / tol
                # relative decay of the oracle residual per cycle around that audit: an error injected
                # every cycle is remembered for about 1/decay cycles
                decay = abs(hist[max(k - 2, 0)] - hist[k - 1]) / tol if k >= 2 else 1.0
                misses.append((t, dg, do, margin, decay))
        if dg == do or audit_every == 1:
            e = pot_err(r["f"][t][None], r["g"][t][None], fo[None], go[None], float(w.eps[t]))[0]
            assert e <= pot_tol, f"lane {t}: potential error {e:.3e} > {pot_tol}"
        if o.status == oracle.DONE:
            # the achieved two-sided residual, evaluated in float64 from the emitted potentials
            rr, rc = oracle.residuals(w.x[t], w.y[t], w.a[t], w.b[t], float(w.eps[t]), r["f"][t], r["g"][t])
            assert max(rr, rc) <= tol * (1 + 5e-3), (t, rr, rc)
            assert r["r_row"][t] <= tol
            assert abs(r["r_row"][t] - rr) <= 2e-2 * tol
    return misses


def miss_allowed(margin, decay, floor):
    """A lane may sit one audit away if the oracle's margin at the disputed audit is below the
    arithmetic's residual error: a floor, or for slowly converging lanes the fp32 exponential
    error 2^-22 accumulated over the ~1/decay cycles the iteration remembers (factor 4 slack)."""
    return margin <= max(floor, 4.0 * 2.0 ** -22 / max(decay, 1e-12))


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
