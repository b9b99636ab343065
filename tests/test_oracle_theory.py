"""Pins of oracle/theory.py: the paper's worked example, its KKT identities and its bounds,
checked on tiny dictionaries where the Euclidean projection can be brute-forced."""
import math
import os

import numpy as np
import pytest

from oracle import theory

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "two_atom_tie.txt")


def _golden_row():
    with open(GOLDEN) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    return [float(x) for x in rows[0]]


def test_two_atom_tie_example_of_appendix_D():
    u1, u2, q, a1, a2, y_star, delta = _golden_row()
    U = np.array([[u1, u2]])
    for eps in (1.0, 0.1, 0.01):
        a = theory.entropic_minimiser(U, np.array([q]), eps)
        assert abs(a[0] - a1) < 1e-12 and abs(a[1] - a2) < 1e-12
    gap, p = theory.support_gap(U, np.array([q]))
    assert abs(p.y[0] - y_star) < 1e-12
    # q lies inside the hull: r* = 0, the active face is the whole segment, the gap is 0
    assert np.allclose(p.r, 0.0) and p.active == (0, 1)
    assert gap == delta
    # outside the hull the nearer vertex is the face and the gap is the distance between atoms
    # times the overshoot: q = 1.5 -> r* = 0.5, <r*, u2 - u1> = 0.5
    gap_out, p_out = theory.support_gap(U, np.array([1.5]))
    assert p_out.active == (1,) and gap_out == pytest.approx(0.5, abs=1e-12)


def _instance(seed, M=7, d=3, scale=3.0):
    rng = np.random.default_rng(seed)
    U = rng.standard_normal((d, M))
    q = scale * rng.standard_normal(d)
    return U, q


def test_projection_is_the_library_least_squares_point():
    """The brute-force KKT point minimises |U a - q| over the simplex: no feasible point drawn at
    random, and no vertex, is closer."""
    rng = np.random.default_rng(7)
    for seed in range(8):
        U, q = _instance(seed)
        p = theory.project_onto_hull(U, q)
        best = np.linalg.norm(p.y - q)
        A = rng.dirichlet(np.ones(U.shape[1]) * 0.3, size=4000)
        assert np.all(np.linalg.norm(A @ U.T - q, axis=1) >= best - 1e-12)
        assert np.all(np.linalg.norm(U.T - q, axis=1) >= best - 1e-12)
        assert abs(p.alpha.sum() - 1) < 1e-12 and np.all(p.alpha >= 0)
        assert np.allclose(U @ p.alpha, p.y)


def test_gap_equals_min_off_face_multiplier():
    """Lemma 1 / Lemma 2: nu* = h_K(r*), mu*_j = h_K(r*) - <r*, u_j>, Delta = min_{j not in I} mu*_j,
    and stationarity U^T (U a* - q) + nu* 1 - mu* = 0 with mu* . a* = 0."""
    for seed in range(10):
        U, q = _instance(seed)
        gap, p = theory.support_gap(U, q)
        h = float((U.T @ p.r).max())
        assert p.nu == pytest.approx(h, abs=1e-10)
        stat = U.T @ (U @ p.alpha - q) + p.nu - p.mu
        assert np.max(np.abs(stat)) < 1e-9
        assert np.max(np.abs(p.mu * p.alpha)) < 1e-9 and np.all(p.mu >= -1e-10)
        off = [j for j in range(U.shape[1]) if j not in p.active]
        assert gap == pytest.approx(min(p.mu[j] for j in off), abs=1e-10)
        assert gap > 0


def test_entropic_minimiser_is_stationary_and_minimal():
    rng = np.random.default_rng(3)
    for seed in range(4):
        U, q = _instance(seed)
        for eps in (0.5, 0.05):
            a = theory.entropic_minimiser(U, q, eps)
            assert abs(a.sum() - 1) < 1e-12 and np.all(a > 0)
            assert theory.stationarity_residual(U, q, eps, a) < 1e-13
            f0 = theory.entropic_objective(U, q, eps, a)
            for _ in range(200):   # strictly convex: every feasible perturbation is worse
                b = np.clip(a + 1e-3 * rng.standard_normal(a.size), 1e-300, None)
                b /= b.sum()
                assert theory.entropic_objective(U, q, eps, b) >= f0 - 1e-15


def test_off_face_weights_obey_corollary_2():
    """For small eps and every off-face atom j:  a_eps,j <= exp(-Delta / (2 eps)), and the off-face
    mass is at most (M - |I|) times that."""
    for seed in range(6):
        U, q = _instance(seed)
        gap, p = theory.support_gap(U, q)
        off = [j for j in range(U.shape[1]) if j not in p.active]
        for frac in (8.0, 16.0):
            eps = gap / frac
            a = theory.entropic_minimiser(U, q, eps)
            bound = math.exp(-gap / (2 * eps))
            assert np.all(a[off] <= bound)
            assert a[off].sum() <= len(off) * bound


def test_main_theorem_shape_linear_on_face_exponential_off_face():
    """|y_eps - y*| is O(eps) when the face has dimension >= 1 (halving eps roughly halves it)
    and exponentially small when the face is a single vertex."""
    seen_vertex = seen_face = False
    for seed in range(30):
        U, q = _instance(seed, M=6, d=2, scale=2.5)
        gap, p = theory.support_gap(U, q)
        if gap < 0.3:
            continue
        e1, e2 = gap / 12, gap / 24
        d1 = np.linalg.norm(U @ theory.entropic_minimiser(U, q, e1) - p.y)
        d2 = np.linalg.norm(U @ theory.entropic_minimiser(U, q, e2) - p.y)
        D = max(np.linalg.norm(U[:, i] - U[:, j]) for i in range(6) for j in range(6))
        if len(p.active) == 1:
            seen_vertex = True
            # only the leakage term remains (Cor. 2 + readout lemma)
            assert d1 <= D * 5 * math.exp(-gap / (2 * e1))
            assert d2 <= D * 5 * math.exp(-gap / (2 * e2))
        elif min(p.alpha[list(p.active)]) > 0.1:
            seen_face = True
            assert 1.6 < d1 / d2 < 2.4
    assert seen_vertex and seen_face


def test_fw_gap_certifies_suboptimality():
    """App. E: f(a_t) - f(a*) <= g_t for any feasible a_t, with equality to 0 at the optimum."""
    rng = np.random.default_rng(5)
    for seed in range(5):
        U, q = _instance(seed)
        p = theory.project_onto_hull(U, q)
        f = lambda a: 0.5 * float(np.sum((U @ a - q) ** 2))
        assert theory.fw_gap(U, q, p.alpha) < 1e-9
        for _ in range(50):
            a = rng.dirichlet(np.ones(U.shape[1]))
            assert f(a) - f(p.alpha) <= theory.fw_gap(U, q, a) + 1e-12
