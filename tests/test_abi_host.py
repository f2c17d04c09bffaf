"""CPU-only checks of the C-ABI library: it builds, loads, exports every entry point the
header declares, and its host-side validation answers with status codes (no GPU needed, no
compute call is made)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2607_24741_b200 import build
    build.build()
    from paper_2607_24741_b200 import binding
    return binding


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(sinkhorn_\w+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(B):
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(B.lib, n), n
    assert names == set(B.EXPORTS) | set(B.EXTRA_EXPORTS)


def test_workspace_size_and_config_validation(B):
    cfg = B.make_config(8, 64, 64, 2, compute="f32")
    small = B.sinkhorn_batch_workspace_bytes(cfg)
    assert small > 0 and small % 256 == 0
    big = B.sinkhorn_batch_workspace_bytes(B.make_config(16, 64, 64, 2, compute="f32"))
    assert big > small
    wide = B.sinkhorn_batch_workspace_bytes(B.make_config(8, 64, 64, 2, compute="f64"))
    assert wide > small
    # an automatic batch may switch to float64 coordinates: it is sized for them
    assert B.sinkhorn_batch_workspace_bytes(B.make_config(8, 64, 64, 2)) == wide
    assert B.sinkhorn_batch_host_workspace_bytes(cfg) > small
    for bad in (B.make_config(0, 64, 64, 2), B.make_config(8, 64, 64, 0), B.make_config(8, 64, 64, 2, max_iter=0),
                B.make_config(8, 64, 64, 2, audit_every=0), B.make_config(8, 64, 64, 2, column_split=5),
                B.make_config(8, 64, 64, 2, mode=7)):
        assert B.sinkhorn_batch_workspace_bytes(bad) == 0


def test_guard_band_and_lane_capacity_show_in_the_workspace(B):
    # host logic only: what the guard band and the lane capacity cost in workspace
    W, n, m = 8, 64, 48
    ws = lambda d, **kw: B.sinkhorn_batch_workspace_bytes(B.make_config(W, n, m, d, compute="f32", **kw))
    lane = lambda pts, d, es: -(-(pts * d * es) // 16) * 16          # a lane's raw cloud, 16-byte aligned
    pad = lambda b: -(-b // 256) * 256                                # an array of the workspace
    # d <= 32: on by default (0), off when negative; the difference is the raw copies of x and y and their two strips
    on, off = ws(2), ws(2, guard_band=-1.0)
    assert on == ws(2, guard_band=1e-3)
    assert on - off == pad(W * lane(n, 2, 4)) + pad(W * lane(m, 2, 4)) + 2 * 256
    # deeper lanes: off unless the caller names a width
    assert ws(64) == ws(64, guard_band=-1.0)
    assert ws(64, guard_band=1e-2) > ws(64)
    assert B.sinkhorn_batch_workspace_bytes(B.make_config(W, n, m, 2, guard_band=0.75)) == 0      # at most 0.5
    # per-lane outputs grow with the capacity, per-slot state does not
    grow = ws(2, lane_capacity=3 * W) - ws(2)
    assert grow >= 2 * W * (n + m) * 8 and grow < 2 * W * (n + m) * 8 + 64 * 1024


def test_create_rejects_bad_arguments_without_touching_the_gpu(B):
    cfg = B.make_config(8, 64, 64, 2)
    h = ctypes.c_void_p()
    one = ctypes.c_void_p(256)
    rc = B.lib.sinkhorn_batch_create(None, one, one, one, one, 1e-3, ctypes.byref(cfg), ctypes.byref(h))
    assert rc == 1 and h.value is None                           # SKB_ERR_NULL
    rc = B.lib.sinkhorn_batch_create(one, one, one, one, one, 0.0, ctypes.byref(cfg), ctypes.byref(h))
    assert rc == 3                                                # tol <= 0
    rc = B.lib.sinkhorn_batch_create(one, one, one, one, one, 1e-3, ctypes.byref(cfg), ctypes.byref(h))
    assert rc == 4 and b"workspace" in B.lib.sinkhorn_batch_last_error(None)
    bad = B.make_config(8, 0, 64, 2)
    rc = B.lib.sinkhorn_batch_create(one, one, one, one, one, 1e-3, ctypes.byref(bad), ctypes.byref(h))
    assert rc == 2
    cfg.workspace = 256 + 8; cfg.workspace_bytes = 1 << 40
    rc = B.lib.sinkhorn_batch_create(one, one, one, one, one, 1e-3, ctypes.byref(cfg), ctypes.byref(h))
    assert rc == 4 and b"aligned" in B.lib.sinkhorn_batch_last_error(None)
    assert B.lib.sinkhorn_batch_step(None, 1) == 1
    B.lib.sinkhorn_batch_destroy(None)                             # no-op
