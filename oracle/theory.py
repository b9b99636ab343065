"""Theory objects on tiny dictionaries (test infrastructure only, numpy fp64).

These are the paper's definitions written out for a handful of atoms, used to pin the
oracle's diagnostics to the statements they come from:

* ``project_onto_hull``   Sec. 4: Euclidean projection y* = Pi_K(q), K = conv(U), residual
                          r* = q - y*, exposed face / active set I (brute force over
                          supports, accepted when the KKT system of Lemma 1 holds).
* ``support_gap``         Def. 1 / Lemma 1: Delta = h_K(r*) - max_{j not in I} <r*, u_j>
                          and the multipliers mu*_j = nu* - <r*, u_j>, nu* = h_K(r*).
* ``entropic_minimiser``  Eq. (5.1): argmin 1/2 |U a - q|^2 + eps * sum a_i log a_i over the
                          simplex, by entropic mirror descent run to a fixed point.
* ``stationarity_residual``  interior KKT of the entropic problem (App. A):
                          a_i proportional to exp(<u_i, q - U a> / eps).
* ``fw_gap``              App. E: Frank-Wolfe duality gap g_t of the unregularised problem.

Columns of ``U`` are atoms (d x M), as in the paper's notation table.
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass
from typing import Tuple

import numpy as np


@dataclass
class Projection:
    y: np.ndarray        # Pi_K(q)
    r: np.ndarray        # q - y
    alpha: np.ndarray    # barycentric weights of y (one optimal choice)
    support: Tuple[int, ...]   # supp(alpha)
    active: Tuple[int, ...]    # I = {i : <r, u_i> = h_K(r)} (vertices on the exposed face)
    nu: float            # h_K(r) = max_i <r, u_i>
    mu: np.ndarray       # mu_j = nu - <r, u_j> >= 0


def _solve_on_support(U: np.ndarray, q: np.ndarray, idx) -> np.ndarray:
    """min 1/2 |U_I a - q|^2  s.t. sum a = 1 (sign-free), via its KKT linear system."""
    UI = U[:, idx]
    k = len(idx)
    A = np.zeros((k + 1, k + 1))
    A[:k, :k] = UI.T @ UI
    A[:k, k] = 1.0
    A[k, :k] = 1.0
    b = np.concatenate([UI.T @ q, [1.0]])
    sol = np.linalg.lstsq(A, b, rcond=None)[0]
    return sol[:k]


def project_onto_hull(U: np.ndarray, q: np.ndarray, tol: float = 1e-10) -> Projection:
    U = np.asarray(U, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    d, M = U.shape
    assert M <= 14, "brute force over supports: tiny dictionaries only"
    for k in range(1, M + 1):
        for idx in itertools.combinations(range(M), k):
            a = _solve_on_support(U, q, list(idx))
            if np.any(a < -tol) or abs(a.sum() - 1.0) > 1e-8:
                continue
            y = U[:, idx] @ a
            r = q - y
            proj = U.T @ r
            nu = float(proj[list(idx)].max())
            # KKT: every atom of the support attains nu, nobody exceeds it
            if np.all(np.abs(proj[list(idx)] - nu) <= tol * (1 + abs(nu))) and np.all(proj <= nu + tol * (1 + abs(nu))):
                alpha = np.zeros(M)
                alpha[list(idx)] = np.clip(a, 0.0, None)
                alpha /= alpha.sum()
                active = tuple(int(i) for i in np.nonzero(np.abs(proj - nu) <= 1e-9 * (1 + abs(nu)))[0])
                return Projection(y, r, alpha, tuple(i for i in idx if a[idx.index(i)] > tol), active, nu, nu - proj)
    raise RuntimeError("no KKT point found")


def support_gap(U: np.ndarray, q: np.ndarray) -> Tuple[float, Projection]:
    """Delta(q) of Def. 1 (= min off-face multiplier, Lemma 1).

    When q lies in the hull (r* = 0, outside the nontrivial regime H1) every atom attains
    h_K(0) = 0 and the paper's convention is Delta = 0 (App. D).  +inf if r* != 0 and every
    atom is active."""
    p = project_onto_hull(U, q)
    if np.linalg.norm(p.r) <= 1e-12 * (1.0 + np.linalg.norm(q)):
        return 0.0, p
    off = [j for j in range(U.shape[1]) if j not in p.active]
    if not off:
        return float("inf"), p
    proj = U.T @ p.r
    return float(p.nu - proj[off].max()), p


def entropic_minimiser(U: np.ndarray, q: np.ndarray, eps: float, tol: float = 1e-14,
                       max_iter: int = 2_000_000) -> np.ndarray:
    """Unique minimiser of Eq. (5.1), by entropic mirror descent in log-coordinates.

    One step solves  min <grad f(a_t), a> + eps*Omega(a) + KL(a || a_t)/eta  exactly:
    log a+ = (log a_t - eta * grad f(a_t)) / (1 + eta*eps) + const.
    """
    U = np.asarray(U, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    M = U.shape[1]
    L = max(float((U * U).sum(axis=0).max()), 1e-12) * 2.0   # relative smoothness of f w.r.t. entropy
    eta = 1.0 / L
    loga = np.full(M, -np.log(M))
    for _ in range(max_iter):
        a = np.exp(loga)
        grad = U.T @ (U @ a - q)
        new = (loga - eta * grad) / (1.0 + eta * eps)
        new -= new.max()
        new -= np.log(np.exp(new).sum())
        done = np.max(np.abs(np.exp(new) - a)) < tol * 1e-2 and stationarity_residual(U, q, eps, np.exp(new)) < tol
        loga = new
        if done:
            break
    return np.exp(loga)


def stationarity_residual(U, q, eps, alpha) -> float:
    """max_i | a_i - softmax(U^T (q - U a) / eps)_i | : zero exactly at the minimiser."""
    U = np.asarray(U, dtype=np.float64)
    z = U.T @ (np.asarray(q, dtype=np.float64) - U @ alpha) / eps
    z -= z.max()
    w = np.exp(z)
    w /= w.sum()
    return float(np.max(np.abs(w - alpha)))


def entropic_objective(U, q, eps, alpha) -> float:
    a = np.asarray(alpha, dtype=np.float64)
    r = np.asarray(U, dtype=np.float64) @ a - np.asarray(q, dtype=np.float64)
    ent = np.sum(np.where(a > 0, a * np.log(np.where(a > 0, a, 1.0)), 0.0))
    return 0.5 * float(r @ r) + eps * float(ent)


def fw_gap(U, q, alpha) -> float:
    """g = <grad f(a), a> - min_j grad f(a)_j  for f(a) = 1/2 |U a - q|^2 (App. E)."""
    U = np.asarray(U, dtype=np.float64)
    grad = U.T @ (U @ alpha - np.asarray(q, dtype=np.float64))
    return float(grad @ alpha - grad.min())
