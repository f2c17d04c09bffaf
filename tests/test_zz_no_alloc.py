"""The allocation-free row-residual entry point against the batch API's own residual.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.  It must pass both alone in a fresh process and after the rest of the suite."""
import numpy as np
import pytest

from paper_2607_24741_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_scratch_residual_matches_the_batch_residual_twice_in_a_row():
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
