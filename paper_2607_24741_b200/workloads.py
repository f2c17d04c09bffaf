"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds input generation only — none of the Sinkhorn arithmetic — so
that the CPU oracle and the CUDA library can both be fed the very same arrays.
Values are drawn in float64 from ``numpy.random.default_rng(SEED0 + index)``
with one child stream per lane, then rounded ONCE to the storage type (fp32, or
bf16 for the feature-coupling workload); the rounded arrays are what both sides
receive.  Marginals are normalised in float64 before the rounding and are not
re-normalised afterwards.

The paper measures on MetroPT-3, Packer19, ImageNet-32 features and LiDAR clips
(workload table in its appendix); none of those can be used here, so these
generators stand in for them with the same shapes, weight laws and cost scales.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SEED0 = 20260724

NAMES = ("tiny", "sensor", "feature", "registration", "sweep")
SWEEP_TOLS = (1e-2, 3e-3, 1e-3, 3e-4, 1e-4)


@dataclass
class Workload:
    name: str
    x: np.ndarray            # [W, n, d] float32 (bf16-representable when xy_dtype == "bf16")
    y: np.ndarray            # [W, m, d] float32
    a: np.ndarray            # [W, n] float32, positive, each lane sums to 1 (to fp32 rounding)
    b: np.ndarray            # [W, m] float32
    eps: np.ndarray          # [W] float32
    tol: float
    max_iter: int
    xy_dtype: str = "f32"    # "f32" | "bf16"
    x_bits: np.ndarray | None = None   # [W, n, d] uint16 bf16 patterns when xy_dtype == "bf16"
    y_bits: np.ndarray | None = None
    meta: dict = field(default_factory=dict)

    @property
    def shape(self):
        W, n, d = self.x.shape
        return W, n, self.y.shape[1], d


def to_bf16_bits(v32: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(v32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def from_bf16_bits(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def _f32(v):
    return np.ascontiguousarray(v, dtype=np.float32)


def _streams(index: int, W: int):
    return np.random.default_rng(SEED0 + index).spawn(W)


def tiny(W=8, n=64, m=None, tol=1e-3, max_iter=5000) -> Workload:
    """Heterogeneous 2-D Gaussians: x~N(0,I), y~N(mu_k, s_k I), uniform weights, eps=0.05."""
    m = n if m is None else m
    d = 2
    x = np.empty((W, n, d)); y = np.empty((W, m, d))
    for k, r in enumerate(_streams(0, W)):
        mu = r.uniform(0.0, 2.0, size=d)
        s = r.uniform(0.5, 2.0)
        x[k] = r.standard_normal((n, d))
        y[k] = mu + np.sqrt(s) * r.standard_normal((m, d))
    a = np.full((W, n), 1.0 / n); b = np.full((W, m), 1.0 / m)
    return Workload("tiny", _f32(x), _f32(y), _f32(a), _f32(b), _f32(np.full(W, 0.05)), tol, max_iter)


def sensor(W=256, n=512, m=None, d=15, tol=1e-3, max_iter=5000) -> Workload:
    """Sensor-window couplings: z-scored features with per-lane drift, Dirichlet(5)
    marginals, eps = 0.1 x the lane's median pairwise squared distance."""
    m = n if m is None else m
    x = np.empty((W, n, d)); y = np.empty((W, m, d))
    a = np.empty((W, n)); b = np.empty((W, m)); eps = np.empty(W)
    for k, r in enumerate(_streams(1, W)):
        delta = 0.3 * r.standard_normal(d)
        u = r.uniform(0.0, 1.0, size=d)
        x[k] = r.standard_normal((n, d))
        y[k] = delta + np.sqrt(1.0 + 0.5 * u) * r.standard_normal((m, d))
        a[k] = r.dirichlet(np.full(n, 5.0)); b[k] = r.dirichlet(np.full(m, 5.0))
    x32, y32 = _f32(x), _f32(y)
    for k in range(W):   # workload parameter: cost scale of the rounded clouds
        xx = x32[k].astype(np.float64); yy = y32[k].astype(np.float64)
        sq = (xx * xx).sum(1)[:, None] + (yy * yy).sum(1)[None, :] - 2.0 * xx @ yy.T
        eps[k] = 0.1 * np.median(sq)
    return Workload("sensor", x32, y32, _f32(a), _f32(b), _f32(eps), tol, max_iter)


def feature(W=64, n=1024, m=None, d=512, classes=10, offset=1.0, tol=1e-3, max_iter=5000) -> Workload:
    """Minibatch feature couplings: L2-normalised class-clustered embeddings stored in
    bf16, uniform weights, eps=0.05."""
    m = n if m is None else m
    x = np.empty((W, n, d), dtype=np.float32); y = np.empty((W, m, d), dtype=np.float32)
    for k, r in enumerate(_streams(2, W)):
        mu = offset * r.standard_normal((classes, d))
        lx = r.integers(0, classes, size=n); ly = r.integers(0, classes, size=m)
        px = r.standard_normal((n, d)) + mu[lx]
        py = r.standard_normal((m, d)) + mu[ly]
        x[k] = px / np.linalg.norm(px, axis=1, keepdims=True)
        y[k] = py / np.linalg.norm(py, axis=1, keepdims=True)
    xb, yb = to_bf16_bits(x), to_bf16_bits(y)
    a = np.full((W, n), 1.0 / n); b = np.full((W, m), 1.0 / m)
    return Workload("feature", from_bf16_bits(xb), from_bf16_bits(yb), _f32(a), _f32(b),
                    _f32(np.full(W, 0.05)), tol, max_iter, "bf16", xb, yb)


def registration(W=32, n=8192, m=None, tol=1e-3, max_iter=5000) -> Workload:
    """Point-cloud registration: noisy unit-sphere sample x, y = rotated x + jitter with
    10% uniform outliers, weights ~ U[0.5,1.5] normalised, eps=0.01.  (m == n here.)"""
    d = 3
    m = n
    x = np.empty((W, n, d)); y = np.empty((W, m, d))
    a = np.empty((W, n)); b = np.empty((W, m))
    for k, r in enumerate(_streams(3, W)):
        v = r.standard_normal((n, d)); v /= np.linalg.norm(v, axis=1, keepdims=True)
        x[k] = v * (1.0 + 0.02 * r.standard_normal((n, 1)))
        q, rr = np.linalg.qr(r.standard_normal((d, d)))
        q = q * np.sign(np.diag(rr))            # Haar-distributed orthogonal matrix
        if np.linalg.det(q) < 0: q[:, 0] = -q[:, 0]
        yy = x[k] @ q.T + 0.01 * r.standard_normal((n, d))
        out = r.random(n) < 0.10
        yy[out] = r.uniform(-1.0, 1.0, size=(int(out.sum()), d))
        y[k] = yy
        wa = r.uniform(0.5, 1.5, size=n); wb = r.uniform(0.5, 1.5, size=m)
        a[k] = wa / wa.sum(); b[k] = wb / wb.sum()
    return Workload("registration", _f32(x), _f32(y), _f32(a), _f32(b), _f32(np.full(W, 0.01)),
                    tol, max_iter)


def sweep(W=1024, n=256, m=None, d=8, tol=1e-3, max_iter=50000) -> Workload:
    """Completion-depth disagreement sweep: Gaussian clouds, uniform weights, eps
    log-uniform in [0.01, 0.5] per lane.  Run once per tolerance in SWEEP_TOLS."""
    m = n if m is None else m
    x = np.empty((W, n, d)); y = np.empty((W, m, d)); eps = np.empty(W)
    for k, r in enumerate(_streams(4, W)):
        x[k] = r.standard_normal((n, d)); y[k] = r.standard_normal((m, d))
        eps[k] = np.exp(r.uniform(np.log(0.01), np.log(0.5)))
    a = np.full((W, n), 1.0 / n); b = np.full((W, m), 1.0 / m)
    return Workload("sweep", _f32(x), _f32(y), _f32(a), _f32(b), _f32(eps), tol, max_iter)


_MAKERS = {"tiny": tiny, "sensor": sensor, "feature": feature, "registration": registration,
           "sweep": sweep}


def make(name: str, **overrides) -> Workload:
    """Build one of the five workloads; keyword overrides (W, n, m, tol, ...) give the
    reduced sizes used by parity tests."""
    return _MAKERS[name](**overrides)
