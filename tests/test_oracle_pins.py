"""Pins for the float64 CPU oracle against what the paper and the mathematics fix.

None of these re-type the oracle's own formulas: they use closed forms, a
scaling-domain iteration with a materialised kernel matrix, library routines
(scipy logsumexp / cdist) on special cases, invariants (Eq. 4, dual ascent,
Eq. 6-8) and the slot counts the paper prints.
"""
import os

import numpy as np
import pytest
from scipy.spatial.distance import cdist
from scipy.special import logsumexp

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def plan(C, f, g, eps):
    return np.exp((f[:, None] + g[None, :] - C) / eps)


def scaling_domain(C, a, b, eps, cycles):
    """Eq. 3 exactly as printed: u <- a/(Kv), v <- b/(K^T u), K materialised."""
    K = np.exp(-C / eps)
    u, v = np.ones_like(a), np.ones_like(b)
    for _ in range(cycles):
        u = a / (K @ v)
        v = b / (K.T @ u)
    return u, v, K


def rand_instance(seed, n, m, d, scale=1.0):
    r = np.random.default_rng(seed)
    x = r.standard_normal((n, d)) * scale
    y = r.standard_normal((m, d)) * scale + 0.3
    a = r.uniform(0.5, 1.5, n); a /= a.sum()
    b = r.uniform(0.5, 1.5, m); b /= b.sum()
    return x, y, a, b


def test_cost_matrix_is_squared_euclidean(oracle):
    x, y, _, _ = rand_instance(1, 7, 5, 3)
    C = oracle.cost_matrix(x, y)
    assert C.shape == (7, 5)
    np.testing.assert_allclose(C, cdist(x, y, "sqeuclidean"), rtol=1e-13, atol=1e-15)
    # a transposed operand or a halved cost would fail these two
    assert C[2, 4] == pytest.approx(((x[2] - y[4]) ** 2).sum(), rel=1e-14)
    assert oracle.cost_matrix(np.zeros((1, 1)), np.full((1, 1), 3.0))[0, 0] == pytest.approx(9.0)


def test_two_by_two_closed_form_in_one_cycle(oracle):
    # a=b=(1/2,1/2), C=[[0,c],[c,0]]: pi = [[1,k],[k,1]]/(2+2k), k=exp(-c/eps), after one cycle
    L, eps = 1.3, 0.7
    x = np.array([[0.0], [L]]); y = np.array([[0.0], [L]])
    a = b = np.array([0.5, 0.5])
    r = oracle.solve_lane(x, y, a, b, eps, 1e-12, fixed_cycles=1)
    kappa = np.exp(-L * L / eps)
    expect = np.array([[1, kappa], [kappa, 1]]) / (2 + 2 * kappa)
    C = np.array([[0, L * L], [L * L, 0.0]])
    np.testing.assert_allclose(plan(C, r.f, r.g, eps), expect, rtol=1e-13)
    assert r.depth == 1 and r.status == oracle.DONE


def test_single_point_lane(oracle):
    r = oracle.solve_lane(np.array([[1.0, 2.0]]), np.array([[4.0, 6.0]]), [1.0], [1.0], 0.3, 1e-9)
    assert r.depth == 1
    assert r.f[0] + r.g[0] == pytest.approx(25.0, rel=1e-14)   # pi = 1 => f + g = C


def test_large_eps_gives_product_plan(oracle):
    x, y, a, b = rand_instance(2, 6, 9, 2)
    C = cdist(x, y, "sqeuclidean")
    for eps in (1e3, 1e6):
        r = oracle.solve_lane(x, y, a, b, eps, 1e-3)
        P = plan(C, r.f, r.g, eps)
        assert r.depth == 1
        assert np.abs(P - np.outer(a, b)).max() < 4 * C.max() / eps * np.outer(a, b).max()


@pytest.mark.parametrize("n,m,d,eps", [(3, 3, 1, 0.5), (5, 8, 2, 0.3), (8, 4, 3, 1.0), (6, 6, 2, 0.1)])
def test_matches_scaling_domain_iteration(oracle, n, m, d, eps):
    x, y, a, b = rand_instance(10 + n + m, n, m, d)
    C = cdist(x, y, "sqeuclidean")
    for cycles in (1, 2, 7):
        r = oracle.solve_lane(x, y, a, b, eps, 1e-300, fixed_cycles=cycles)
        u, v, K = scaling_domain(C, a, b, eps, cycles)
        np.testing.assert_allclose(r.f, eps * np.log(u), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(r.g, eps * np.log(v), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(plan(C, r.f, r.g, eps), u[:, None] * K * v[None, :], rtol=1e-10)


def test_converged_plan_is_the_unique_optimum(oracle):
    # run to r <= 1e-13: exact marginals + Gibbs form = KKT point of the strictly convex Eq. 1
    x, y, a, b = rand_instance(5, 6, 7, 2)
    eps = 0.4
    C = cdist(x, y, "sqeuclidean")
    r = oracle.solve_lane(x, y, a, b, eps, 1e-13, max_iter=200000)
    assert r.status == oracle.DONE
    P = plan(C, r.f, r.g, eps)
    assert np.abs(P.sum(1) - a).sum() <= 1e-13 and np.abs(P.sum(0) - b).sum() <= 1e-13
    primal = (C * P).sum() + eps * (P * (np.log(P) - 1)).sum()
    dual = a @ r.f + b @ r.g - eps * P.sum()
    assert primal == pytest.approx(dual, abs=1e-11)
    # any feasible perturbation (keeps both marginals) must not lower the primal
    rng = np.random.default_rng(0)
    for _ in range(20):
        i, k = rng.choice(6, 2, replace=False); j, l = rng.choice(7, 2, replace=False)
        Q = P.copy(); t = 1e-3 * min(P[i, j], P[k, l], P[i, l], P[k, j])
        Q[i, j] += t; Q[k, l] += t; Q[i, l] -= t; Q[k, j] -= t
        assert (C * Q).sum() + eps * (Q * (np.log(Q) - 1)).sum() >= primal - 1e-15


def test_legs_against_library_logsumexp(oracle):
    x, y, a, b = rand_instance(7, 9, 11, 3)
    C = cdist(x, y, "sqeuclidean")
    eps = 0.2
    g = np.random.default_rng(3).standard_normal(11)
    f = oracle.f_leg(C, g, a, eps)
    np.testing.assert_allclose(f, eps * (np.log(a) - logsumexp((g[None, :] - C) / eps, axis=1)), rtol=1e-13)
    g2 = oracle.g_leg(C, f, b, eps)
    np.testing.assert_allclose(g2, eps * (np.log(b) - logsumexp((f[:, None] - C) / eps, axis=0)), rtol=1e-13)


def test_updated_marginal_is_current_after_each_leg(oracle):
    # Eq. 4: after the g-leg the column marginal is b; after the f-leg the row marginal is a
    x, y, a, b = rand_instance(8, 12, 10, 2)
    C = cdist(x, y, "sqeuclidean")
    eps = 0.15
    g = np.zeros(10)
    for _ in range(5):
        f = oracle.f_leg(C, g, a, eps)
        row, col = oracle.marginals(C, f, g, eps)
        assert np.abs(row - a).sum() <= 1e-13
        assert np.abs(col - b).sum() > 1e-6          # the other side is genuinely off
        g = oracle.g_leg(C, f, b, eps)
        row, col = oracle.marginals(C, f, g, eps)
        assert np.abs(col - b).sum() <= 1e-13
        assert np.abs(row - a).sum() > 1e-8


def test_dual_ascent_and_unit_mass(oracle):
    x, y, a, b = rand_instance(9, 16, 12, 2)
    eps = 0.1
    r = oracle.solve_lane(x, y, a, b, eps, 1e-6, dual=True, history=True, max_iter=20000)
    D = r.dual_hist[: 2 * r.depth]
    assert np.all(np.diff(D) >= -1e-13)               # block coordinate ascent
    C = cdist(x, y, "sqeuclidean")
    # total mass is 1 after any half-step, so D = <a,f> + <b,g> - eps
    assert D[-1] == pytest.approx(a @ r.f + b @ r.g - eps, abs=1e-12)
    assert oracle.dual_value(C, r.f, r.g, eps, a, b) == pytest.approx(D[-1], abs=1e-13)
    P = plan(C, r.f, r.g, eps)
    primal = (C * P).sum() + eps * (P * (np.log(P) - 1)).sum()
    assert primal == pytest.approx(D[-1], abs=1e-5)   # gap closes at the fixed point


def test_depth_is_first_audit_that_passes_and_residual_decays(oracle):
    x, y, a, b = rand_instance(11, 24, 24, 2)
    eps, tol = 0.05, 1e-3
    r = oracle.solve_lane(x, y, a, b, eps, tol, history=True, neighbours=True)
    two = np.maximum(r.hist_row[: r.depth], r.hist_col[: r.depth])
    assert two[-1] <= tol and np.all(two[:-1] > tol)
    assert r.r_row == r.hist_row[r.depth - 1] and r.r_col == r.hist_col[r.depth - 1]
    assert np.all(np.diff(r.hist_row[: r.depth]) <= 1e-15)   # L1 residual non-increasing
    assert r.r_col <= 1e-13
    # neighbours really are one cycle either side
    p = oracle.solve_lane(x, y, a, b, eps, tol, fixed_cycles=r.depth - 1)
    q = oracle.solve_lane(x, y, a, b, eps, tol, fixed_cycles=r.depth + 1)
    np.testing.assert_array_equal(p.f, r.f_prev); np.testing.assert_array_equal(q.g, r.g_next)
    assert q.depth == r.depth                                  # fixed run reports the same first pass
    # independent residual from the plan definition
    C = cdist(x, y, "sqeuclidean"); P = plan(C, r.f, r.g, eps)
    assert np.abs(P.sum(1) - a).sum() == pytest.approx(r.r_row, rel=1e-10)


def test_audit_grid_and_iteration_limit(oracle):
    x, y, a, b = rand_instance(12, 16, 16, 2)
    r1 = oracle.solve_lane(x, y, a, b, 0.05, 1e-3)
    r4 = oracle.solve_lane(x, y, a, b, 0.05, 1e-3, audit_every=4)
    assert r4.depth % 4 == 0 and r1.depth <= r4.depth < r1.depth + 4
    lim = oracle.solve_lane(x, y, a, b, 0.05, 1e-3, max_iter=max(1, r1.depth - 1))
    assert lim.status == oracle.ITER_LIMIT and lim.depth == r1.depth - 1 and lim.r_row > 1e-3
    # the screen can only delay a release, never authorise one
    s = oracle.solve_lane(x, y, a, b, 0.05, 1e-3, tol_screen=5e-4)
    assert s.depth >= r1.depth and s.r_row <= 5e-4


def test_cost_and_eps_scale_together(oracle):
    # C -> 2C with eps -> 2 eps leaves the plan and the depth unchanged and doubles the potentials;
    # a hidden factor 1/2 in the cost, or eps applied on one leg only, breaks this with eps fixed
    x, y, a, b = rand_instance(13, 10, 14, 3)
    r = oracle.solve_lane(x, y, a, b, 0.2, 1e-4)
    s = oracle.solve_lane(x * np.sqrt(2), y * np.sqrt(2), a, b, 0.4, 1e-4)
    assert r.depth == s.depth
    np.testing.assert_allclose(2 * r.f, s.f, rtol=1e-9, atol=1e-12)
    t = oracle.solve_lane(x + 5.0, y + 5.0, a, b, 0.2, 1e-4)      # translation invariance
    assert t.depth == r.depth
    np.testing.assert_allclose(t.g, r.g, rtol=1e-8, atol=1e-10)


def test_batch_equals_lane_by_lane(oracle):
    # Eq. 2: packing commutes with the per-lane map
    W, n, m, d = 5, 12, 9, 2
    xs, ys, As, Bs = zip(*[rand_instance(20 + t, n, m, d) for t in range(W)])
    eps = np.array([0.05, 0.1, 0.2, 0.5, 1.0])
    B = oracle.solve_batch(np.stack(xs), np.stack(ys), np.stack(As), np.stack(Bs), eps, 1e-3, threads=3)
    assert 1 <= B.threads <= 3
    for t in range(W):
        r = oracle.solve_lane(xs[t], ys[t], As[t], Bs[t], eps[t], 1e-3)
        assert r.depth == B.depth[t]
        np.testing.assert_array_equal(r.f, B.f[t]); np.testing.assert_array_equal(r.g, B.g[t])
    lmax = int(B.depth.max())
    S = oracle.solve_batch(np.stack(xs), np.stack(ys), np.stack(As), np.stack(Bs), eps, 1e-3,
                           fixed_cycles=lmax)
    np.testing.assert_array_equal(S.depth, B.depth)               # same first-pass depths
    assert np.all(S.r_row <= 1e-3)                                # every lane still passes at l_max
    k = int(np.argmax(B.depth)); np.testing.assert_array_equal(S.f[k], B.f[k])


def test_slot_identity_and_paper_counts(oracle):
    rng = np.random.default_rng(4)
    for _ in range(50):
        depths = rng.integers(1, 40, size=rng.integers(1, 30))
        s = oracle.slot_counts(depths)
        assert s["S_active"] == depths.sum()                       # Eq. 7
        assert s["S_static"] == depths.size * depths.max()
        assert s["R"] == s["S_static"] - s["S_active"]             # Eq. 8
        assert (s["R"] == 0) == bool(np.all(depths == depths[0]))   # Proposition 2
        A = s["widths"]
        assert A[0] == depths.size and np.all(np.diff(A) <= 0)
    for line in open(os.path.join(GOLD, "paper_slot_counts.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, W, s_static, s_active, audit = line.split()
        W, s_static, s_active, audit = int(W), int(s_static), int(s_active), int(audit)
        lmax = s_static // W
        assert lmax * W == s_static and lmax % audit == 0           # slot = lane x cycle on the audit grid
        # build a depth profile on the audit grid with that maximum and that total
        depths = np.full(W, lmax); deficit = s_static - s_active; t = 1
        while deficit > 0:
            cut = min(deficit, lmax - audit) // audit * audit
            if cut == 0:
                break
            depths[t] -= cut; deficit -= cut; t += 1
        s = oracle.slot_counts(depths)
        assert s["S_static"] == s_static and s["S_active"] == s_static - (s_static - s_active - deficit)
        assert s["R"] == s_static - s["S_active"]


def test_warm_proposal_is_the_same_iteration_started_later(oracle):
    # Section "Initialization and repeated couplings": a proposal only replaces the starting point.
    # Starting from the cold iteration's own state after j cycles must land on the cold run's states
    # j cycles earlier (semigroup property of the fixed map F_t of Eq. 2) - checked against the cold
    # run, not against the warm code path itself.
    x, y, a, b = rand_instance(11, 9, 12, 2)
    eps, tol = 0.2, 1e-7
    cold = oracle.solve_lane(x, y, a, b, eps, tol)
    assert cold.depth > 6
    for j in (1, 4):
        part = oracle.solve_lane(x, y, a, b, eps, tol, fixed_cycles=j)
        warm = oracle.solve_lane(x, y, a, b, eps, tol, f0=part.f, g0=part.g)
        assert warm.depth == cold.depth - j and warm.status == oracle.DONE
        np.testing.assert_allclose(warm.f, cold.f, rtol=0, atol=1e-14)
        np.testing.assert_allclose(warm.g, cold.g, rtol=0, atol=1e-14)
    # zeros given explicitly are the cold proposal
    z = oracle.solve_lane(x, y, a, b, eps, tol, f0=np.zeros(9), g0=np.zeros(12))
    assert z.depth == cold.depth and np.array_equal(z.f, cold.f)


def test_audit_of_the_proposal_is_eq5_at_the_proposal(oracle):
    x, y, a, b = rand_instance(12, 7, 10, 3)
    eps = 0.3
    C = cdist(x, y, "sqeuclidean")
    conv = oracle.solve_lane(x, y, a, b, eps, 1e-12)
    g0 = conv.g + 0.01 * np.sin(np.arange(10))
    P = plan(C, conv.f, g0, eps)
    rr, rc = np.abs(P.sum(1) - a).sum(), np.abs(P.sum(0) - b).sum()
    assert rr > 1e-3 and rc > 1e-3                        # neither marginal is current for this proposal
    # thresholds above both residuals: the proposal passes as it is, depth 0, nothing is updated
    r0 = oracle.solve_lane(x, y, a, b, eps, 2 * max(rr, rc), f0=conv.f, g0=g0, audit_initial=True)
    assert r0.depth == 0 and r0.status == oracle.DONE
    assert r0.r_row == pytest.approx(rr, rel=1e-12) and r0.r_col == pytest.approx(rc, rel=1e-12)
    np.testing.assert_array_equal(r0.f, conv.f); np.testing.assert_array_equal(r0.g, g0)
    # stop threshold between the two residuals, screen wide open: the two-sided test must fail on the larger one
    lo, hi = min(rr, rc), max(rr, rc)
    r1 = oracle.solve_lane(x, y, a, b, eps, 0.5 * (lo + hi), tol_screen=10.0, f0=conv.f, g0=g0, audit_initial=True)
    assert r1.depth >= 1
    # without the initial audit the same call never reports depth 0
    r2 = oracle.solve_lane(x, y, a, b, eps, 2 * max(rr, rc), f0=conv.f, g0=g0)
    assert r2.depth == 1


def test_plan_application_against_the_two_by_two_plan_and_the_marginals(oracle):
    # a=b=(1/2,1/2), C=[[0,c],[c,0]]: the plan after one cycle is [[1,k],[k,1]]/(2+2k) (closed form above)
    L, eps = 1.3, 0.7
    x = np.array([[0.0], [L]]); y = np.array([[0.0], [L]])
    a = b = np.array([0.5, 0.5])
    r = oracle.solve_lane(x, y, a, b, eps, 1e-12, fixed_cycles=1)
    kappa = np.exp(-L * L / eps)
    v = np.array([[2.0, -1.0], [0.5, 3.0]])
    expect = (np.array([[1, kappa], [kappa, 1]]) / (2 + 2 * kappa)) @ v
    np.testing.assert_allclose(oracle.apply_plan(x, y, eps, r.f, r.g, v), expect, rtol=1e-13)
    # applied to ones it is the row marginal; applied to y it is a_i times the barycentric image
    x, y, a, b = rand_instance(21, 9, 7, 3)
    s = oracle.solve_lane(x, y, a, b, 0.4, 1e-10)
    row, _ = oracle.marginals(oracle.cost_matrix(x, y), s.f, s.g, 0.4)
    np.testing.assert_allclose(oracle.apply_plan(x, y, 0.4, s.f, s.g, np.ones((7, 1)))[:, 0], row, rtol=1e-13)
    T = oracle.apply_plan(x, y, 0.4, s.f, s.g, y) / a[:, None]
    assert np.all(T.min(0) >= y.min(0) - 1e-9) and np.all(T.max(0) <= y.max(0) + 1e-9)   # convex combinations of y
