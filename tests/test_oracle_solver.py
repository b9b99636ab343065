"""Pins of oracle/solver.py (entropic mirror descent on the candidate set, Sec. 7 step 3 / Eq. (5.1) /
App. E): what the mathematics fixes about the iterates, checked against code that does not share
the solver's update (the pinned minimiser and KKT residual of oracle/theory.py, a library softmax,
finite differences, brute force over the simplex vertices)."""

import numpy as np
import pytest
import scipy.special

import oracle
from oracle import solver, theory
from util import geometry, host_arrays
from workloads import WorkloadSpec, make_workload


def _instance(seed, n=9, d=5, scale=2.0):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((d, n)), scale * rng.standard_normal(d)


def test_zero_iterations_is_the_library_softmax_of_the_scores():
    for seed in range(5):
        U, q = _instance(seed)
        for eps in (0.3, 2.0):
            sol = solver.entropic_mirror_descent(U, q, eps, 0)
            assert np.allclose(sol.alpha, scipy.special.softmax(U.T @ q / eps), rtol=0, atol=1e-15)
            assert len(sol.trace) == 1


def test_iterates_descend_and_reach_the_pinned_minimiser():
    """f_eps never increases along the iterates (relative smoothness with eta = 1/L), and the limit is
    the unique minimiser: the interior KKT residual vanishes and the weights agree with the
    independently started, differently stepped solver of oracle/theory.py."""
    for seed in range(6):
        U, q = _instance(seed)
        for eps in (0.5, 0.1):
            sol = solver.entropic_mirror_descent(U, q, eps, 400)
            f = [theory.entropic_objective(U, q, eps, a) for a in sol.trace]
            assert all(f[i + 1] <= f[i] + 1e-13 for i in range(len(f) - 1))
            assert f[0] - f[-1] > 1e-5        # the closed-form start is not the minimiser
            long = solver.entropic_mirror_descent(U, q, eps, 60000)
            assert theory.stationarity_residual(U, q, eps, long.alpha) < 1e-11
            assert np.max(np.abs(long.alpha - theory.entropic_minimiser(U, q, eps))) < 1e-9
            assert long.objective == pytest.approx(theory.entropic_objective(U, q, eps, long.alpha), abs=1e-12)


def test_every_iterate_is_interior_and_normalised():
    U, q = _instance(11, n=14, d=4, scale=6.0)
    sol = solver.entropic_mirror_descent(U, q, 0.05, 6)
    for a in sol.trace:
        assert abs(a.sum() - 1.0) < 1e-12 and np.all(a >= 0) and np.all(np.isfinite(a))


def test_scaling_invariance_pins_the_step_and_the_place_of_epsilon():
    """(U, q, eps) -> (cU, cq, c^2 eps) multiplies f_eps by c^2 and must leave every iterate unchanged
    (eta scales by 1/c^2).  A step that ignored L, or an eps applied on the wrong side, breaks this."""
    U, q = _instance(3)
    a = solver.entropic_mirror_descent(U, q, 0.4, 6)
    for c in (0.25, 7.0):
        b = solver.entropic_mirror_descent(c * U, c * q, c * c * 0.4, 6)
        assert b.step == pytest.approx(a.step / (c * c), rel=1e-12)
        for x, y in zip(a.trace, b.trace):
            assert np.max(np.abs(x - y)) < 1e-12
        assert b.objective == pytest.approx(c * c * a.objective, rel=1e-10)
        assert b.fw_gap == pytest.approx(c * c * a.fw_gap, rel=1e-9, abs=1e-12)


def test_identical_atoms_keep_uniform_weights():
    """All candidates equal: the gradient is a constant vector, the weights stay uniform."""
    u = np.array([[1.0], [-2.0], [0.5]])
    U = np.repeat(u, 6, axis=1)
    sol = solver.entropic_mirror_descent(U, np.array([0.3, 0.1, -1.0]), 0.7, 5)
    for a in sol.trace:
        assert np.allclose(a, 1.0 / 6.0, atol=1e-15)
    assert sol.fw_gap == pytest.approx(0.0, abs=1e-12)


def test_fw_gap_is_the_max_over_vertices_and_bounds_the_suboptimality():
    """App. E: g = max_j <grad f(a), a - e_j>, with the gradient taken by central differences here;
    and f(a) - min f <= g, the minimum taken from the brute-force projection."""
    for seed in range(5):
        U, q = _instance(seed, n=7, d=3, scale=3.0)
        sol = solver.entropic_mirror_descent(U, q, 0.2, 3)
        a = sol.alpha
        f = lambda x: 0.5 * float(np.sum((U @ x - q) ** 2))
        h = 1e-6
        grad = np.array([(f(a + h * e) - f(a - h * e)) / (2 * h) for e in np.eye(a.size)])
        brute = max(float(grad @ (a - e)) for e in np.eye(a.size))
        assert sol.fw_gap == pytest.approx(brute, abs=1e-6)
        assert sol.fw_gap == pytest.approx(theory.fw_gap(U, q, a), abs=1e-12)
        fstar = f(theory.project_onto_hull(U, q).alpha)
        assert f(a) - fstar <= sol.fw_gap + 1e-12
        assert sol.residual2 == pytest.approx(2 * f(a), rel=1e-12)


def test_more_iterations_move_towards_the_minimiser_geometrically():
    """eps-strong convexity relative to the entropy: KL(a* || a_t) contracts by at least
    1 / (1 + eta * eps) per iteration."""
    U, q = _instance(8)
    eps = 0.6
    astar = theory.entropic_minimiser(U, q, eps)
    sol = solver.entropic_mirror_descent(U, q, eps, 30)
    kl = [float(np.sum(astar * (np.log(astar) - np.log(a)))) for a in sol.trace]
    rate = 1.0 / (1.0 + sol.step * eps)
    assert all(kl[i + 1] <= rate * kl[i] + 1e-14 for i in range(len(kl) - 1))


def _small_workload():
    spec = WorkloadSpec(name="t", config=9, batch=2, n_q_heads=4, n_kv_heads=2, P=3, K_c=20,
                        seq_lens=(150, 70), needles=2, needle_positions="uniform")
    return make_workload(spec, seed=77)


def test_sparse_entropic_on_a_paged_cache():
    """Zero iterations reproduce the closed-form pass of the oracle; with iterations the output stays a
    convex combination of the SAME candidates' value rows, every unit's objective does not increase,
    and the candidates, gap diagnostics and fallback flags are those of the closed-form pass."""
    w = _small_workload()
    q, K, V, bt, sl = host_arrays(w)
    g = geometry(w)
    summ = oracle.build_summaries(g, K, bt, sl)
    rt = oracle.route(g, q, summ, bt, sl, w.spec.P)
    r0 = solver.sparse_entropic(g, q, K, V, bt, sl, rt.pages, w.spec.K_c, w.epsilon, w.gap_threshold, 0)
    assert np.max(np.abs(r0.out - r0.base.out)) < 1e-12
    assert np.max(np.abs(r0.alpha - r0.base.cand_weight)) < 1e-12
    prev = r0
    for iters in (2, 6):
        r = solver.sparse_entropic(g, q, K, V, bt, sl, rt.pages, w.spec.K_c, w.epsilon, w.gap_threshold, iters)
        assert np.array_equal(r.base.cand_pos, r0.base.cand_pos) and np.array_equal(r.base.fallback, r0.base.fallback)
        assert np.allclose(r.alpha.sum(-1), 1.0, atol=1e-12) and np.all(r.alpha >= 0)
        assert np.all((r.alpha > 0) == (r0.base.cand_pos >= 0))
        assert np.all(r.objective <= prev.objective + 1e-9)
        assert np.all(r.fw_gap >= -1e-9)
        prev = r
    # the weights moved: the quadratic term pushes mass away from the closed-form weights
    assert np.max(np.abs(prev.alpha - r0.alpha)) > 1e-6
