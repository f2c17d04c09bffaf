"""The allocation-free row-residual entry point.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.  It must pass both alone in a fresh process and after the rest of the suite."""
import numpy as np
import pytest

from paper_2607_24741_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_scratch_residual_matches_the_batch_residual_twice_in_a_row(oracle):
    import torch
    from paper_2607_24741_b200 import binding as B
    dev = torch.device("cuda:0")
    t = lambda v: torch.from_numpy(v).to(dev)
    for w in (wl.make("sensor", W=12, n=300, m=260), wl.make("tiny")):
        x, y, a, b, eps = t(w.x), t(w.y), t(w.a), t(w.b), t(w.eps)
        sb = B.SinkhornBatch(x, y, a, b, eps, w.tol, max_iter=w.max_iter)
        sb.drain()
        f, g = sb.potentials(f64=True)
        r_ref, _ = sb.residuals()                      # existing entry point: row residual at retirement
        sb.close()
        first = B.sinkhorn_row_residual_static(x, y, a, f, g, eps)
        second = B.sinkhorn_row_residual_static(x, y, a, f, g, eps)   # same shared scratch again
        torch.cuda.synchronize()
        r_ref = r_ref.cpu().numpy(); first = first.cpu().numpy(); second = second.cpu().numpy()
        assert np.all(r_ref <= w.tol) and np.all(r_ref > 0)
        # same tolerance as the parity suite's residual check: 2% of the stopping tolerance
        assert np.abs(first - r_ref).max() <= 2e-2 * w.tol
        np.testing.assert_array_equal(first, second)
        # and against the oracle's float64 row residual of the same potentials (both are float64
        # evaluations of the same sum; the result is returned as float32)
        fh, gh = f.cpu().numpy(), g.cpu().numpy()
        for k in range(w.shape[0]):
            rr, _ = oracle.residuals(w.x[k], w.y[k], w.a[k], w.b[k], float(w.eps[k]), fh[k], gh[k])
            assert abs(first[k] - rr) <= 1e-6 * rr + 1e-12


def test_static_scratch_at_its_limits_allocates_nothing(oracle):
    # the largest shapes the fixed array serves: 64 row blocks per lane (n = 8192) and 256 lanes; after a
    # warm-up call the free device memory must not move across further calls
    import torch
    from paper_2607_24741_b200 import binding as B
    dev = torch.device("cuda:0")
    t = lambda v: torch.from_numpy(v).to(dev)
    rng = np.random.default_rng(3)
    big = wl.make("registration", W=2, n=8192)
    wide = wl.make("sweep", W=256, n=40, m=24)
    cases = []
    for w in (big, wide):
        W, n, m, d = w.shape
        f = (0.05 * rng.standard_normal((W, n))).astype(np.float64)
        g = (0.05 * rng.standard_normal((W, m)) - 1.0).astype(np.float64)     # plan mass well below 1: no overflow anywhere
        cases.append((w, f, g, [t(w.x), t(w.y), t(w.a), torch.from_numpy(f).to(dev), torch.from_numpy(g).to(dev), t(w.eps)]))
    B.sinkhorn_row_residual_static(*cases[1][3]); torch.cuda.synchronize()      # warm-up: module load, address look-up
    outs = [torch.empty(c[0].shape[0], dtype=torch.float32, device=dev) for c in cases]
    free0 = torch.cuda.mem_get_info(dev)[0]
    for rep in range(2):
        for (w, f, g, args), out in zip(cases, outs):
            W, n, m, d = w.shape
            rc = B.lib.sinkhorn_row_residual_static(*[a.data_ptr() for a in args], W, n, m, d, out.data_ptr(),
                                                    torch.cuda.current_stream(dev).cuda_stream)
            assert rc == 0 and B.lib.sinkhorn_row_residual_static_last_error() == b""
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info(dev)[0] == free0
    for (w, f, g, args), out in zip(cases, outs):
        got = out.cpu().numpy()
        for k in (0, w.shape[0] - 1):
            rr, _ = oracle.residuals(w.x[k], w.y[k], w.a[k], w.b[k], float(w.eps[k]), f[k], g[k])
            assert abs(got[k] - rr) <= 1e-6 * rr


def test_static_scratch_limits_are_reported():
    import torch
    from paper_2607_24741_b200 import binding as B
    z = torch.zeros(1, dtype=torch.float32, device="cuda:0")
    zd = torch.zeros(1, dtype=torch.float64, device="cuda:0")
    rc = B.lib.sinkhorn_row_residual_static(z.data_ptr(), z.data_ptr(), z.data_ptr(), zd.data_ptr(), zd.data_ptr(),
                                            z.data_ptr(), 257, 4, 4, 2, z.data_ptr(), None)
    assert rc == 2 and b"256 lanes" in B.lib.sinkhorn_row_residual_static_last_error()
    rc = B.lib.sinkhorn_row_residual_static(z.data_ptr(), z.data_ptr(), z.data_ptr(), zd.data_ptr(), zd.data_ptr(),
                                            z.data_ptr(), 1, 8193, 4, 2, z.data_ptr(), None)
    assert rc == 2
