"""ctypes binding of libsinkhorn_batch.so — argument marshalling only.

Every step of the solve runs in the library's CUDA kernels; PyTorch supplies
device memory and the stream.  There is no fallback: if the shared library is
missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsinkhorn_batch.so")

SKB_OK = 0
STATUS_NAMES = {0: "SKB_OK", 1: "SKB_ERR_NULL", 2: "SKB_ERR_SHAPE", 3: "SKB_ERR_VALUE",
                4: "SKB_ERR_WORKSPACE", 5: "SKB_ERR_STATE", 6: "SKB_ERR_CUDA"}
MODES = {"active": 0, "masked": 1, "static": 2, "masked_exit": 3}
COMPUTE = {"auto": 0, "f32": 1, "mixed": 2, "f64": 3, "tensor": 4}
LANE_RUNNING, LANE_DONE, LANE_ITER_LIMIT, LANE_NONFINITE = 0, 1, 2, 3

EXPORTS = (
    "sinkhorn_batch_workspace_bytes", "sinkhorn_batch_create", "sinkhorn_batch_step",
    "sinkhorn_batch_drain", "sinkhorn_batch_active", "sinkhorn_batch_potentials",
    "sinkhorn_batch_potentials_f64", "sinkhorn_batch_depths", "sinkhorn_batch_residuals",
    "sinkhorn_batch_stats", "sinkhorn_batch_destroy", "sinkhorn_batch_last_error",
    "sinkhorn_batch_host_workspace_bytes", "sinkhorn_batch_solve_host",
    "sinkhorn_batch_launch_count", "sinkhorn_batch_profile_update", "sinkhorn_batch_arithmetic",
    "sinkhorn_batch_selftest_bounded_wait", "sinkhorn_batch_warm_start", "sinkhorn_batch_set_profiling",
    "sinkhorn_batch_cycle_trace", "sinkhorn_batch_selftest_unit_rates", "sinkhorn_batch_last_audit",
    "sinkhorn_batch_refill", "sinkhorn_batch_apply_plan", "sinkhorn_batch_check_guards",
)
PHASES = ("create", "f_leg", "column_check", "plan", "emit_move", "g_leg")
# entry points outside the sinkhorn_batch_* family
EXTRA_EXPORTS = ("sinkhorn_row_residual_static", "sinkhorn_row_residual_static_last_error")


class SkbConfig(ctypes.Structure):
    _fields_ = [("W", ctypes.c_int), ("n", ctypes.c_int), ("m", ctypes.c_int), ("d", ctypes.c_int),
                ("xy_dtype", ctypes.c_int), ("mode", ctypes.c_int), ("compute", ctypes.c_int),
                ("max_iter", ctypes.c_int), ("audit_every", ctypes.c_int),
                ("tol_screen", ctypes.c_float), ("column_split", ctypes.c_int),
                ("cost_form", ctypes.c_int),
                ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t), ("guard_band", ctypes.c_float),
                ("lane_capacity", ctypes.c_int)]


class SkbError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{STATUS_NAMES.get(code, code)}: {msg}")
        self.code = code


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_24741_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, cfgp = ctypes.c_void_p, ctypes.POINTER(SkbConfig)
    lib.sinkhorn_batch_workspace_bytes.restype = ctypes.c_size_t
    lib.sinkhorn_batch_workspace_bytes.argtypes = [cfgp]
    lib.sinkhorn_batch_host_workspace_bytes.restype = ctypes.c_size_t
    lib.sinkhorn_batch_host_workspace_bytes.argtypes = [cfgp]
    lib.sinkhorn_batch_create.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, cfgp, ctypes.POINTER(vp)]
    lib.sinkhorn_batch_step.argtypes = [vp, ctypes.c_int]
    lib.sinkhorn_batch_drain.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
    lib.sinkhorn_batch_active.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
    lib.sinkhorn_batch_potentials.argtypes = [vp, vp, vp]
    lib.sinkhorn_batch_potentials_f64.argtypes = [vp, vp, vp]
    lib.sinkhorn_batch_depths.argtypes = [vp, vp, vp]
    lib.sinkhorn_batch_residuals.argtypes = [vp, vp, vp]
    lib.sinkhorn_batch_stats.argtypes = [vp, ctypes.POINTER(ctypes.c_longlong), ctypes.POINTER(ctypes.c_int),
                                         vp, ctypes.c_int, ctypes.POINTER(ctypes.c_longlong),
                                         ctypes.POINTER(ctypes.c_float)]
    lib.sinkhorn_batch_last_audit.argtypes = [vp, vp, vp, vp]
    lib.sinkhorn_batch_apply_plan.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int, vp]
    lib.sinkhorn_batch_refill.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
    lib.sinkhorn_batch_warm_start.argtypes = [vp, vp, vp, ctypes.c_int]
    lib.sinkhorn_batch_set_profiling.argtypes = [vp, ctypes.c_int]
    lib.sinkhorn_batch_cycle_trace.argtypes = [vp, vp, ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
    lib.sinkhorn_batch_selftest_bounded_wait.argtypes = [vp, ctypes.c_float, vp]
    lib.sinkhorn_batch_check_guards.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
    lib.sinkhorn_batch_selftest_unit_rates.argtypes = [ctypes.POINTER(ctypes.c_double), vp, vp]
    lib.sinkhorn_batch_arithmetic.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
    lib.sinkhorn_batch_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_longlong)]
    lib.sinkhorn_batch_profile_update.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_float)]
    lib.sinkhorn_batch_destroy.argtypes = [vp]
    lib.sinkhorn_batch_destroy.restype = None
    lib.sinkhorn_batch_last_error.argtypes = [vp]
    lib.sinkhorn_batch_last_error.restype = ctypes.c_char_p
    lib.sinkhorn_batch_solve_host.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, cfgp, vp, vp, vp, vp, vp, vp,
                                              ctypes.POINTER(ctypes.c_longlong), ctypes.POINTER(ctypes.c_int)]
    lib.sinkhorn_row_residual_static.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_int, ctypes.c_int,
                                                 ctypes.c_int, ctypes.c_int, vp, vp]
    lib.sinkhorn_row_residual_static.restype = ctypes.c_int
    lib.sinkhorn_row_residual_static_last_error.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("sinkhorn_batch_workspace_bytes", "sinkhorn_batch_host_workspace_bytes",
                        "sinkhorn_batch_destroy", "sinkhorn_batch_last_error"):
            getattr(lib, name).restype = ctypes.c_int
    return lib


lib = _load()


def _check(code, handle=None):
    if code != SKB_OK:
        msg = lib.sinkhorn_batch_last_error(handle)
        raise SkbError(code, msg.decode() if msg else "")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def make_config(W, n, m, d, *, bf16=False, mode="active", compute="auto", max_iter=5000,
                audit_every=1, tol_screen=0.0, column_split=0, cost_form=0, stream=0, guard_band=0.0,
                lane_capacity=0) -> SkbConfig:
    return SkbConfig(W, n, m, d, 1 if bf16 else 0, MODES[mode] if isinstance(mode, str) else mode,
                     COMPUTE[compute] if isinstance(compute, str) else compute, max_iter, audit_every,
                     tol_screen, column_split, cost_form, stream, None, 0, guard_band, lane_capacity)


# ---- functions with the C names ------------------------------------------------------

def sinkhorn_batch_workspace_bytes(cfg: SkbConfig) -> int:
    return lib.sinkhorn_batch_workspace_bytes(ctypes.byref(cfg))


def sinkhorn_batch_host_workspace_bytes(cfg: SkbConfig) -> int:
    return lib.sinkhorn_batch_host_workspace_bytes(ctypes.byref(cfg))


def sinkhorn_batch_create(x, y, a, b, eps, tol, cfg: SkbConfig):
    h = ctypes.c_void_p()
    _check(lib.sinkhorn_batch_create(_ptr(x), _ptr(y), _ptr(a), _ptr(b), _ptr(eps), tol, ctypes.byref(cfg),
                                     ctypes.byref(h)))
    return h


def sinkhorn_batch_step(h, cycles):
    _check(lib.sinkhorn_batch_step(h, cycles), h)


def sinkhorn_batch_drain(h) -> int:
    c = ctypes.c_int(0)
    _check(lib.sinkhorn_batch_drain(h, ctypes.byref(c)), h)
    return c.value


def sinkhorn_batch_active(h) -> int:
    c = ctypes.c_int(0)
    _check(lib.sinkhorn_batch_active(h, ctypes.byref(c)), h)
    return c.value


def sinkhorn_batch_destroy(h):
    lib.sinkhorn_batch_destroy(h)


def sinkhorn_row_residual_static(x, y, a, f, g, eps, stream=None):
    """Row residual of potentials (f, g) per lane, with no workspace and no allocation inside the
    library (see the header for limits and the sharing rule).  x, y, a, eps: float32 CUDA tensors;
    f, g: float64.  Returns the library's status code and writes into the tensor it returns."""
    W, n, d = x.shape
    m = y.shape[1]
    out = torch.empty(W, dtype=torch.float32, device=x.device)
    st = (stream or torch.cuda.current_stream(x.device)).cuda_stream
    rc = lib.sinkhorn_row_residual_static(_ptr(x), _ptr(y), _ptr(a), _ptr(f), _ptr(g), _ptr(eps), W, n, m, d,
                                          _ptr(out), st)
    if rc != SKB_OK:
        raise SkbError(rc, lib.sinkhorn_row_residual_static_last_error().decode())
    return out


def unit_rates(device=None):
    """Measured operations per second of the fp32 FMA, packed fp32x2 FMA, float64 FMA and fp32 ex2
    units (the library's self-test loops)."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    sink = torch.zeros(1, dtype=torch.float32, device=dev)
    out = (ctypes.c_double * 4)()
    with torch.cuda.device(dev):
        _check(lib.sinkhorn_batch_selftest_unit_rates(out, _ptr(sink), torch.cuda.current_stream(dev).cuda_stream))
    return dict(zip(("ffma", "ffma2", "dfma", "ex2"), list(out)))


class SinkhornBatch:
    """One batch of W lanes on the current CUDA device (thin wrapper over the C calls)."""

    def __init__(self, x, y, a, b, eps, tol, *, mode="active", compute="auto", max_iter=5000,
                 audit_every=1, tol_screen=0.0, column_split=0, cost_form=0, stream=None, guard_band=0.0,
                 lane_capacity=0):
        if not (x.is_cuda and y.is_cuda and a.is_cuda and b.is_cuda and eps.is_cuda):
            raise ValueError("x, y, a, b, eps must be CUDA tensors")
        if x.dtype not in (torch.float32, torch.bfloat16) or y.dtype != x.dtype:
            raise ValueError("x and y must both be float32 or both be bfloat16")
        for t in (a, b, eps):
            if t.dtype != torch.float32:
                raise ValueError("a, b, eps must be float32")
        x, y, a, b, eps = (t.contiguous() for t in (x, y, a, b, eps))
        W, n, d = x.shape
        m = y.shape[1]
        if y.shape != (W, m, d) or a.shape != (W, n) or b.shape != (W, m) or eps.shape != (W,):
            raise ValueError("shapes must be x[W,n,d] y[W,m,d] a[W,n] b[W,m] eps[W]")
        self.W, self.n, self.m, self.d = W, n, m, d
        self.device = x.device
        self.stream = stream if stream is not None else torch.cuda.current_stream(x.device)
        self.cfg = make_config(W, n, m, d, bf16=x.dtype == torch.bfloat16, mode=mode, compute=compute,
                               max_iter=max_iter, audit_every=audit_every, tol_screen=tol_screen,
                               column_split=column_split, cost_form=cost_form, stream=self.stream.cuda_stream,
                               guard_band=guard_band, lane_capacity=lane_capacity)
        self.L = max(W, lane_capacity)
        need = sinkhorn_batch_workspace_bytes(self.cfg)
        if need == 0:
            raise SkbError(2, "configuration rejected (unsupported shape or bad option)")
        self.workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
        self.cfg.workspace = self.workspace.data_ptr()
        self.cfg.workspace_bytes = need
        self._keep = (x, y, a, b, eps)
        self.h = None
        with torch.cuda.device(x.device):
            self.h = sinkhorn_batch_create(x, y, a, b, eps, float(tol), self.cfg)

    def step(self, cycles=1):
        sinkhorn_batch_step(self.h, cycles)

    def drain(self) -> int:
        return sinkhorn_batch_drain(self.h)

    def active(self) -> int:
        return sinkhorn_batch_active(self.h)

    def potentials(self, f64=False):
        dt = torch.float64 if f64 else torch.float32
        f = torch.zeros(self.L, self.n, dtype=dt, device=self.device)
        g = torch.zeros(self.L, self.m, dtype=dt, device=self.device)
        fn = lib.sinkhorn_batch_potentials_f64 if f64 else lib.sinkhorn_batch_potentials
        _check(fn(self.h, _ptr(f), _ptr(g)), self.h)
        return f, g

    def depths(self):
        depth = torch.zeros(self.L, dtype=torch.int32, device=self.device)
        status = torch.zeros(self.L, dtype=torch.int32, device=self.device)
        _check(lib.sinkhorn_batch_depths(self.h, _ptr(depth), _ptr(status)), self.h)
        return depth, status

    def residuals(self):
        rr = torch.zeros(self.L, dtype=torch.float32, device=self.device)
        rc = torch.zeros(self.L, dtype=torch.float32, device=self.device)
        _check(lib.sinkhorn_batch_residuals(self.h, _ptr(rr), _ptr(rc)), self.h)
        return rr, rc

    def warm_start(self, f0=None, g0=None, audit_initial=False):
        for t, shape in ((f0, (self.W, self.n)), (g0, (self.W, self.m))):
            if t is not None and (t.dtype != torch.float64 or not t.is_cuda or tuple(t.shape) != shape
                                  or not t.is_contiguous()):
                raise ValueError("f0 [W,n] and g0 [W,m] must be contiguous float64 CUDA tensors")
        _check(lib.sinkhorn_batch_warm_start(self.h, _ptr(f0), _ptr(g0), 1 if audit_initial else 0), self.h)
        self._warm = (f0, g0)

    def check_guards(self) -> int:
        """Index of the first damaged guard strip of the workspace, -1 if all are intact (synchronises)."""
        bad = ctypes.c_int(-2)
        _check(lib.sinkhorn_batch_check_guards(self.h, ctypes.byref(bad)), self.h)
        return bad.value

    def last_audit(self):
        """Row screen value, column residual (NaN where not checked) and screen flag of the most recent audit."""
        rr = torch.full((self.L,), float("nan"), dtype=torch.float32, device=self.device)
        rc = torch.full((self.L,), float("nan"), dtype=torch.float32, device=self.device)
        fl = torch.full((self.L,), -1, dtype=torch.int32, device=self.device)
        _check(lib.sinkhorn_batch_last_audit(self.h, _ptr(rr), _ptr(rc), _ptr(fl)), self.h)
        return rr, rc, fl

    def refill(self, x, y, a, b, eps) -> int:
        """New problems into the slots finished lanes have freed; returns their first lane number."""
        x, y, a, b, eps = (t.contiguous() for t in (x, y, a, b, eps))
        count = x.shape[0]
        if tuple(x.shape) != (count, self.n, self.d) or tuple(y.shape) != (count, self.m, self.d) or \
                tuple(a.shape) != (count, self.n) or tuple(b.shape) != (count, self.m) or tuple(eps.shape) != (count,):
            raise ValueError("shapes must be x[c,n,d] y[c,m,d] a[c,n] b[c,m] eps[c]")
        first = ctypes.c_int(-1)
        _check(lib.sinkhorn_batch_refill(self.h, _ptr(x), _ptr(y), _ptr(a), _ptr(b), _ptr(eps), count, ctypes.byref(first)), self.h)
        self._keep = self._keep + (x, y, a, b, eps)
        return first.value

    def apply_plan(self, v):
        """out[t, i, :] = sum_j pi_ij v[t, j, :] with the plan of the finished lanes; v [W, m, dv] float32."""
        x, y, _a, _b, eps = self._keep[:5]
        v = v.contiguous()
        if v.dtype != torch.float32 or v.dim() != 3 or tuple(v.shape[:2]) != (self.W, self.m):
            raise ValueError("v must be float32 [W, m, dv]")
        out = torch.empty(self.W, self.n, v.shape[2], dtype=torch.float32, device=self.device)
        _check(lib.sinkhorn_batch_apply_plan(self.h, _ptr(x), _ptr(y), _ptr(eps), _ptr(v), v.shape[2], _ptr(out)), self.h)
        return out

    def set_profiling(self, on=True):
        _check(lib.sinkhorn_batch_set_profiling(self.h, 1 if on else 0), self.h)

    def stats(self, widths_cap=0):
        slots, terms, cycles = ctypes.c_longlong(0), ctypes.c_longlong(0), ctypes.c_int(0)
        buf = (ctypes.c_int * max(widths_cap, 1))()
        ph = (ctypes.c_float * len(PHASES))()
        _check(lib.sinkhorn_batch_stats(self.h, ctypes.byref(slots), ctypes.byref(cycles),
                                        ctypes.cast(buf, ctypes.c_void_p), widths_cap, ctypes.byref(terms), ph), self.h)
        k = min(cycles.value, widths_cap)
        return {"slots": slots.value, "cycles": cycles.value, "pair_terms": terms.value,
                "widths": list(buf[:k]), "phase_ms": dict(zip(PHASES, list(ph)))}

    def cycle_trace(self):
        n = ctypes.c_int(0)
        _check(lib.sinkhorn_batch_cycle_trace(self.h, None, 0, ctypes.byref(n)), self.h)
        buf = (ctypes.c_float * max(n.value, 1))()
        _check(lib.sinkhorn_batch_cycle_trace(self.h, ctypes.cast(buf, ctypes.c_void_p), n.value, ctypes.byref(n)), self.h)
        return list(buf[:n.value])

    def arithmetic(self) -> str:
        c = ctypes.c_int(0)
        _check(lib.sinkhorn_batch_arithmetic(self.h, ctypes.byref(c)), self.h)
        return {v: k for k, v in COMPUTE.items()}[c.value]

    def launch_count(self) -> int:
        c = ctypes.c_longlong(0)
        _check(lib.sinkhorn_batch_launch_count(self.h, ctypes.byref(c)), self.h)
        return c.value

    def profile_update(self, leg=0, reps=10) -> float:
        ms = ctypes.c_float(0)
        _check(lib.sinkhorn_batch_profile_update(self.h, leg, reps, ctypes.byref(ms)), self.h)
        return ms.value

    def close(self):
        if self.h is not None:
            sinkhorn_batch_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
