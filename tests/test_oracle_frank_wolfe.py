"""Pins of the oracle's Frank-Wolfe solve on a candidate set (orc_frank_wolfe, App. E): textbook
properties of Frank-Wolfe with exact line search, checked against the brute-force projection of
oracle/theory.py, a closed form for two atoms, and an independently written fp64 run of the rule."""
import numpy as np
import pytest
import torch

import oracle
from oracle import theory
from util import geometry, host_arrays
from workloads import WorkloadSpec, make_workload


def _tiny(M, seed, q_scale=1.0):
    """One sequence of M tokens, one head: the dictionary is the M key rows (d = 128)."""
    spec = WorkloadSpec(name="t", config=9, batch=1, n_q_heads=1, n_kv_heads=1, P=1, K_c=M, seq_lens=(M,), needles=0)
    w = make_workload(spec, seed=seed)
    if q_scale != 1.0:
        w.q = (w.q.float() * q_scale).to(torch.bfloat16)
    return w


def _run(w, iters, order=None):
    q, K, V, bt, sl = host_arrays(w)
    M = int(sl[0])
    cp = np.full((1, 1, M), -1, np.int32)
    cp[0, 0] = np.arange(M) if order is None else order
    return oracle.frank_wolfe(geometry(w), q, K, bt, cp, iters), cp


def _dictionary(w):
    q, K, V, bt, sl = host_arrays(w)
    M = int(sl[0])
    Kf = oracle.bf16_to_f32(K).astype(np.float64)
    rows = np.concatenate([Kf[int(bt[0, l]), 0] for l in range((M + 15) // 16)])[:M]
    return rows.T, oracle.bf16_to_f32(q).astype(np.float64)[0, 0]      # U: d x M, q


def test_objective_descends_gap_bounds_suboptimality_and_iterates_stay_sparse():
    for seed in range(4):
        w = _tiny(7, 20 + seed, q_scale=0.3)          # a short query: the projection lies on a proper face
        U, q = _dictionary(w)
        f = lambda a: 0.5 * float(np.sum((U @ a - q) ** 2))
        fstar = f(theory.project_onto_hull(U, q).alpha)
        prev = np.inf
        for iters in (0, 1, 2, 3, 5, 8, 20):
            r, _ = _run(w, iters)
            a = r.alpha[0, 0].astype(np.float64)
            assert abs(a.sum() - 1.0) < 1e-5 and np.all(a >= 0)
            assert np.count_nonzero(a) <= iters + 1
            assert f(a) <= prev + 1e-4
            prev = f(a)
            assert float(r.objective[0, 0]) == pytest.approx(f(a), rel=1e-4, abs=1e-4)
            assert float(r.residual2[0, 0]) == pytest.approx(2 * f(a), rel=1e-4, abs=1e-4)
            # App. E: f(a_t) - f* <= g_t (fp32 slack), and g_t is the gap formula at a_t
            assert f(a) - fstar <= float(r.fw_gap[0, 0]) + 1e-3
            assert float(r.fw_gap[0, 0]) == pytest.approx(theory.fw_gap(U, q, a), rel=1e-3, abs=2e-3)
        long, _ = _run(w, 3000)
        assert f(long.alpha[0, 0].astype(np.float64)) - fstar < 2e-2 * max(1.0, fstar)


def test_two_atoms_reach_the_segment_projection_in_one_step():
    """Textbook: with two atoms one exact-line-search step from the better vertex lands on the projection
    of q onto the segment, a = clamp(<q - u_start, u_other - u_start> / |u_other - u_start|^2, 0, 1)."""
    for seed, scale in ((30, 0.2), (31, 0.5), (32, 3.0)):
        w = _tiny(2, seed, q_scale=scale)
        U, q = _dictionary(w)
        r, _ = _run(w, 1)
        s = U.T @ q
        i0 = int(np.argmax(s))
        d = U[:, 1 - i0] - U[:, i0]
        gamma = float(np.clip((q - U[:, i0]) @ d / (d @ d), 0.0, 1.0))
        want = np.zeros(2)
        want[i0], want[1 - i0] = 1 - gamma, gamma
        assert np.max(np.abs(r.alpha[0, 0] - want)) < 1e-5
        assert float(r.step[0, 0]) == pytest.approx(gamma, abs=1e-5)
        r2, _ = _run(w, 2)                      # already optimal: a second step changes nothing measurable
        assert np.max(np.abs(r2.alpha[0, 0] - r.alpha[0, 0])) < 1e-4


def test_agrees_with_an_fp64_run_of_the_same_rule():
    for seed in range(3):
        w = _tiny(9, 40 + seed, q_scale=0.4)
        U, q = _dictionary(w)
        s = U.T @ q
        a = np.zeros(9)
        a[int(np.argmax(s))] = 1.0
        for _ in range(6):
            y = U @ a
            g = U.T @ y - s
            j = int(np.argmin(g))
            d = U[:, j] - y
            gamma = float(np.clip((q - y) @ d / (d @ d), 0.0, 1.0)) if d @ d > 0 else 0.0
            a = (1 - gamma) * a
            a[j] += gamma
        r, _ = _run(w, 6)
        assert np.max(np.abs(r.alpha[0, 0] - a)) < 1e-4


def test_ties_go_to_the_lower_position_whatever_the_listing_order():
    w = _tiny(6, 50, q_scale=0.3)
    k = w.k_cache.clone()
    page = int(w.block_table[0, 0])
    k[page, 0, 4] = k[page, 0, 1]               # tokens 1 and 4 are the same atom
    w.k_cache = k
    a_fwd, cp_f = _run(w, 8)
    a_rev, cp_r = _run(w, 8, order=np.arange(6)[::-1].copy())
    by_pos_f = np.zeros(6)
    by_pos_f[cp_f[0, 0]] = a_fwd.alpha[0, 0]
    by_pos_r = np.zeros(6)
    by_pos_r[cp_r[0, 0]] = a_rev.alpha[0, 0]
    assert np.array_equal(by_pos_f, by_pos_r)               # the listing order does not matter, bit for bit
    assert by_pos_f[4] == 0.0                               # the duplicate at the higher position is never chosen


def test_zero_iterations_is_the_best_scoring_vertex():
    w = _tiny(10, 60)
    U, q = _dictionary(w)
    r, _ = _run(w, 0)
    assert r.alpha[0, 0][int(np.argmax(U.T @ q))] == 1.0 and r.alpha[0, 0].sum() == 1.0
    assert float(r.step[0, 0]) == 0.0
