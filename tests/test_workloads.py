"""The seeded input generators: shapes, laws and determinism (no Sinkhorn arithmetic here)."""
import numpy as np

from paper_2607_24741_b200 import workloads as wl


def test_shapes_and_weight_laws():
    t = wl.make("tiny")
    assert t.shape == (8, 64, 64, 2) and t.x.dtype == np.float32 and np.all(t.a == np.float32(1 / 64))
    s = wl.make("sensor", W=4, n=96)
    assert s.shape == (4, 96, 96, 15) and np.all(s.a > 0) and np.all(s.b > 0)
    np.testing.assert_allclose(s.a.astype(np.float64).sum(1), 1.0, atol=1e-6)
    assert np.all(s.eps > 1.0) and np.all(s.eps < 8.0)          # 0.1 x median of a ~chi2 cost
    r = wl.make("registration", W=2, n=256)
    assert r.shape == (2, 256, 256, 3)
    inl = np.abs(np.linalg.norm(r.x, axis=2) - 1.0)
    assert np.median(inl) < 0.03 and np.all(r.eps == np.float32(0.01))
    np.testing.assert_allclose(r.b.astype(np.float64).sum(1), 1.0, atol=1e-6)
    assert r.a.max() / r.a.min() <= 3.0 + 1e-6
    w = wl.make("sweep", W=64, n=32)
    assert w.shape == (64, 32, 32, 8) and w.eps.min() >= 0.01 and w.eps.max() <= 0.5 and w.max_iter == 50000


def test_feature_is_bf16_exact_and_normalised():
    f = wl.make("feature", W=2, n=64, d=128)
    assert f.xy_dtype == "bf16" and f.x_bits.dtype == np.uint16
    np.testing.assert_array_equal(wl.from_bf16_bits(f.x_bits), f.x)
    np.testing.assert_array_equal(wl.to_bf16_bits(f.y), f.y_bits)      # already representable
    assert np.all(np.abs(np.linalg.norm(f.x.astype(np.float64), axis=2) - 1) < 4e-3)
    v = np.array([1.0, 1.00390625, 1.01171875, -3.0e38, 1e-40], dtype=np.float32)
    got = wl.from_bf16_bits(wl.to_bf16_bits(v))
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == np.float32(1.015625)   # ties to even


def test_deterministic_and_lane_prefix_stable():
    a = wl.make("sensor", W=3, n=64)
    b = wl.make("sensor", W=3, n=64)
    np.testing.assert_array_equal(a.x, b.x); np.testing.assert_array_equal(a.eps, b.eps)
    c = wl.make("sensor", W=5, n=64)
    np.testing.assert_array_equal(c.y[:3], a.y)                 # one child stream per lane
    assert not np.array_equal(wl.make("tiny").x[0], wl.make("tiny").x[1])
