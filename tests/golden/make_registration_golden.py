"""Writes tests/golden/registration_n8192.npz: the float64 CPU oracle's results for a few lanes
of the point-cloud registration workload at its full size (n = m = 8192, d = 3).

One lane takes the oracle a quarter of an hour or more (a dense 8192 x 8192 cost matrix and
several hundred cycles of Eq. 3 with the audit of Eq. 5 after each), which is too slow for a
test run, so the expected values are computed once by this script and stored.  The script
calls only the oracle and the seeded input generator; nothing it stores comes from the CUDA
path.  Run from the repository root:

    python tests/golden/make_registration_golden.py

Lanes already present in the stored file are kept as they are and only the missing ones of LANES
are computed (the oracle is deterministic, so a full recomputation gives the same file).

The remaining lanes of the workload (LIGHT_LANES) are stored too, with the same fields under keys
prefixed `light_`, their potentials subsampled to every STRIDE-th point, so that the depth of every
lane of the workload is held to the oracle's without the file growing by a quarter of a megabyte
per lane.

Stored per lane t of LANES (arrays are stacked in that order):
    depth, status            completion depth l_t and lane status (Eq. 6)
    r_row, r_col             residuals at the depth (Eq. 5)
    f, g                     float64 potentials at the depth
    f_prev, g_prev           potentials one cycle earlier (float32: used only to compare a lane
    f_next, g_next           that stops one audit away) and one cycle later
    hist                     max(r_row, r_col) at the last HIST audits up to the depth
"""
from __future__ import annotations

import os
import sys
from multiprocessing import Pool

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

LANES = (0, 3, 7, 10, 13, 16, 19, 22, 25, 28, 29, 31)
LIGHT_LANES = tuple(t for t in range(32) if t not in LANES)
STRIDE = 8
HIST = 8
OUT = os.path.join(HERE, "registration_n8192.npz")
POTENTIALS = ("f", "g", "f_prev", "g_prev", "f_next", "g_next")


def _one(t):
    import oracle
    from paper_2607_24741_b200 import workloads as wl
    w = wl.make("registration")
    o = oracle.solve_lane(w.x[t], w.y[t], w.a[t], w.b[t], float(w.eps[t]), w.tol, max_iter=w.max_iter,
                          neighbours=True, history=True)
    h = np.maximum(o.hist_row, o.hist_col)[:o.depth]
    tail = np.full(HIST, np.nan)
    tail[HIST - min(HIST, h.size):] = h[-HIST:]
    print(f"lane {t}: depth {o.depth} status {o.status} r_row {o.r_row:.6e} r_col {o.r_col:.3e}", flush=True)
    return dict(depth=o.depth, status=o.status, r_row=o.r_row, r_col=o.r_col, f=o.f, g=o.g,
                f_prev=o.f_prev.astype(np.float32), g_prev=o.g_prev.astype(np.float32),
                f_next=o.f_next.astype(np.float32), g_next=o.g_next.astype(np.float32), hist=tail)


def _light(r):
    return {k: (np.asarray(v)[::STRIDE] if k in POTENTIALS else v) for k, v in r.items()}


def main():
    import oracle
    oracle.build()
    have, have_light = {}, {}
    if os.path.exists(OUT):
        old = np.load(OUT)
        meta = ("lanes", "n", "tol", "light_lanes", "stride")
        for i, t in enumerate(old["lanes"].tolist()):
            have[t] = {k: old[k][i] for k in old.files if k not in meta and not k.startswith("light_")}
        if "light_lanes" in old.files and int(old["stride"]) == STRIDE:
            for i, t in enumerate(old["light_lanes"].tolist()):
                have_light[t] = {k[6:]: old[k][i] for k in old.files if k.startswith("light_") and k != "light_lanes"}
    todo = [t for t in LANES if t not in have] + [t for t in LIGHT_LANES if t not in have_light and t not in have]
    if todo:
        with Pool(min(len(todo), 6)) as pool:
            for t, r in zip(todo, pool.map(_one, todo, chunksize=1)):
                if t in LANES:
                    have[t] = r
                else:
                    have_light[t] = _light(r)
    for t in LIGHT_LANES:
        if t not in have_light:
            have_light[t] = _light(have[t])          # a lane that used to be stored in full
    res = [have[t] for t in LANES]
    stack = {k: np.stack([np.asarray(r[k]) for r in res]) for k in res[0]}
    lres = [have_light[t] for t in LIGHT_LANES]
    stack.update({"light_" + k: np.stack([np.asarray(r[k]) for r in lres]) for k in lres[0]})
    np.savez_compressed(OUT, lanes=np.array(LANES, np.int32), light_lanes=np.array(LIGHT_LANES, np.int32),
                        stride=np.int32(STRIDE), n=np.int32(8192), tol=np.float64(1e-3), **stack)
    print("wrote", OUT, os.path.getsize(OUT), "bytes")


if __name__ == "__main__":
    main()
