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
HIST = 8
OUT = os.path.join(HERE, "registration_n8192.npz")


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


def main():
    import oracle
    oracle.build()
    have = {}
    if os.path.exists(OUT):
        old = np.load(OUT)
        for i, t in enumerate(old["lanes"].tolist()):
            have[t] = {k: old[k][i] for k in old.files if k not in ("lanes", "n", "tol")}
    todo = [t for t in LANES if t not in have]
    if todo:
        with Pool(min(len(todo), 6)) as pool:
            for t, r in zip(todo, pool.map(_one, todo)):
                have[t] = r
    res = [have[t] for t in LANES]
    stack = {k: np.stack([np.asarray(r[k]) for r in res]) for k in res[0]}
    np.savez_compressed(OUT, lanes=np.array(LANES, np.int32), n=np.int32(8192), tol=np.float64(1e-3), **stack)
    print("wrote", OUT, os.path.getsize(OUT), "bytes")


if __name__ == "__main__":
    main()
