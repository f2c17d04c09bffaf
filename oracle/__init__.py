"""Float64 CPU oracle for batched log-domain Sinkhorn — TEST INFRASTRUCTURE.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It wraps ``sinkhorn_oracle.c`` (plain C, float64, one lane
at a time) through ctypes and adds the depth-profile accounting of the paper's
Proposition 1 (Eq. 6-8).  It shares nothing with the CUDA library and never
imports it.

Parity pins live in ``tests/test_oracle_pins.py``; the completion depth of a
generic instance is "parity unpinned" (the paper prints no depth for a
reproducible input) beyond the structural pins listed there.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import sys
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sinkhorn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

RUNNING, DONE, ITER_LIMIT, NONFINITE = 0, 1, 2, 3

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP over lanes only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True, stdout=sys.stderr, stderr=sys.stderr)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_lane.restype = ctypes.c_int
        _lib.orc_batch.restype = ctypes.c_int
        _lib.orc_dual.restype = ctypes.c_double
        _lib.orc_marginals.restype = ctypes.c_double
    return _lib


def _d(a):
    return None if a is None else a.ctypes.data_as(_dp)


def _c64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


@dataclass
class LaneResult:
    f: np.ndarray
    g: np.ndarray
    depth: int
    status: int
    r_row: float
    r_col: float
    f_prev: np.ndarray | None = None
    g_prev: np.ndarray | None = None
    f_next: np.ndarray | None = None
    g_next: np.ndarray | None = None
    hist_row: np.ndarray | None = None
    hist_col: np.ndarray | None = None
    dual_hist: np.ndarray | None = None


def cost_matrix(x, y) -> np.ndarray:
    """C_ij = |x_i - y_j|^2 through the C routine (difference form)."""
    x, y = _c64(x), _c64(y)
    n, d = x.shape
    m = y.shape[0]
    C = np.empty((n, m))
    _load().orc_cost_matrix(n, m, d, _d(x), _d(y), _d(C))
    return C


def f_leg(C, g, a, eps) -> np.ndarray:
    C, g, a = _c64(C), _c64(g), _c64(a)
    n, m = C.shape
    f = np.empty(n)
    _load().orc_f_leg(n, m, _d(C), _d(g), _d(a), ctypes.c_double(eps), _d(f))
    return f


def g_leg(C, f, b, eps) -> np.ndarray:
    C, f, b = _c64(C), _c64(f), _c64(b)
    n, m = C.shape
    g = np.empty(m)
    _load().orc_g_leg(n, m, _d(C), _d(f), _d(b), ctypes.c_double(eps), _d(g))
    return g


def marginals(C, f, g, eps):
    C, f, g = _c64(C), _c64(f), _c64(g)
    n, m = C.shape
    row, col = np.empty(n), np.empty(m)
    _load().orc_marginals(n, m, _d(C), _d(f), _d(g), ctypes.c_double(eps), _d(row), _d(col))
    return row, col


def residuals(x, y, a, b, eps, f, g):
    """Two-sided L1 residuals (Eq. 5) of the plan defined by potentials (f, g)."""
    C = cost_matrix(x, y)
    row, col = marginals(C, f, g, eps)
    return float(np.abs(row - _c64(a)).sum()), float(np.abs(col - _c64(b)).sum())


def apply_plan(x, y, eps, f, g, v) -> np.ndarray:
    """The plan of Eq. 3, pi = exp((f + g - C)/eps), applied to values v [m, dv]: pi @ v, written out
    from the definition with the dense plan (float64)."""
    C = cost_matrix(x, y)
    pi = np.exp((_c64(f)[:, None] + _c64(g)[None, :] - C) / float(eps))
    return pi @ _c64(v)


def dual_value(C, f, g, eps, a, b) -> float:
    C, f, g, a, b = _c64(C), _c64(f), _c64(g), _c64(a), _c64(b)
    n, m = C.shape
    row, col = np.empty(n), np.empty(m)
    return float(_load().orc_dual(n, m, _d(C), _d(f), _d(g), ctypes.c_double(eps), _d(a), _d(b),
                                  _d(row), _d(col)))


def solve_lane(x, y, a, b, eps, tol, *, tol_screen=0.0, max_iter=5000, audit_every=1,
               fixed_cycles=0, neighbours=False, history=False, dual=False, f0=None, g0=None,
               audit_initial=False) -> LaneResult:
    """Run one lane to its completion depth (or ``fixed_cycles`` cycles), from the cold
    proposal f = g = 0 or from the warm proposal (f0, g0); with ``audit_initial`` the proposal
    itself is audited first and a lane that already passes has depth 0."""
    x, y, a, b = _c64(x), _c64(y), _c64(a), _c64(b)
    f0 = None if f0 is None else _c64(f0)
    g0 = None if g0 is None else _c64(g0)
    n, d = x.shape
    m = y.shape[0]
    f, g = np.empty(n), np.empty(m)
    fp = gp = fn = gn = hr = hc = dh = None
    if neighbours:
        fp, gp, fn, gn = np.empty(n), np.empty(m), np.empty(n), np.empty(m)
    L = fixed_cycles if fixed_cycles > 0 else max_iter
    if history:
        hr, hc = np.full(L, np.nan), np.full(L, np.nan)
    if dual:
        dh = np.full(2 * L, np.nan)
    depth, status = ctypes.c_int(0), ctypes.c_int(0)
    rr, rc = ctypes.c_double(0), ctypes.c_double(0)
    ret = _load().orc_lane(n, m, d, _d(x), _d(y), _d(a), _d(b), ctypes.c_double(float(eps)),
                           ctypes.c_double(float(tol_screen)), ctypes.c_double(float(tol)),
                           int(max_iter), int(audit_every), int(fixed_cycles), _d(f), _d(g),
                           _d(fp), _d(gp), _d(fn), _d(gn), ctypes.byref(depth),
                           ctypes.byref(status), ctypes.byref(rr), ctypes.byref(rc), _d(hr),
                           _d(hc), _d(dh), _d(f0), _d(g0), int(bool(audit_initial)))
    if ret != 0:
        raise ValueError(f"oracle rejected the lane (code {ret})")
    return LaneResult(f, g, depth.value, status.value, rr.value, rc.value, fp, gp, fn, gn, hr, hc, dh)


@dataclass
class BatchResult:
    f: np.ndarray
    g: np.ndarray
    depth: np.ndarray
    status: np.ndarray
    r_row: np.ndarray
    r_col: np.ndarray
    threads: int


def solve_batch(x, y, a, b, eps, tol, *, tol_screen=0.0, max_iter=5000, audit_every=1,
                fixed_cycles=0, threads=0) -> BatchResult:
    """Solve W lanes independently, one whole lane per host thread (Eq. 2)."""
    x, y, a, b = _c64(x), _c64(y), _c64(a), _c64(b)
    W, n, d = x.shape
    m = y.shape[1]
    eps = _c64(np.broadcast_to(np.asarray(eps, dtype=np.float64), (W,)))
    f, g = np.empty((W, n)), np.empty((W, m))
    depth, status = np.zeros(W, np.int32), np.zeros(W, np.int32)
    rr, rc = np.empty(W), np.empty(W)
    used = _load().orc_batch(W, n, m, d, _d(x), _d(y), _d(a), _d(b), _d(eps),
                             ctypes.c_double(float(tol_screen)), ctypes.c_double(float(tol)),
                             int(max_iter), int(audit_every), int(fixed_cycles), int(threads),
                             _d(f), _d(g), depth.ctypes.data_as(_ip), status.ctypes.data_as(_ip),
                             _d(rr), _d(rc))
    if used < 0:
        raise ValueError(f"oracle rejected the batch (code {used})")
    return BatchResult(f, g, depth, status, rr, rc, used)


# ---- depth-profile accounting (Proposition 1, Eq. 6-8) ---------------------

def survivor_widths(depths) -> np.ndarray:
    """A_k = |{t : l_t >= k}| for k = 1..l_max (Eq. 6)."""
    depths = np.asarray(depths, dtype=np.int64)
    lmax = int(depths.max()) if depths.size else 0
    return np.array([(depths >= k).sum() for k in range(1, lmax + 1)], dtype=np.int64)


def slot_counts(depths) -> dict:
    """S_active = sum_k A_k, S_static = W*l_max, R = S_static - sum_t l_t (Eq. 7-8)."""
    depths = np.asarray(depths, dtype=np.int64)
    A = survivor_widths(depths)
    s_static = int(depths.size * (depths.max() if depths.size else 0))
    return {"S_active": int(A.sum()), "S_static": s_static,
            "R": s_static - int(depths.sum()), "widths": A}
