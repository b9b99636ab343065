"""Iterative entropic solve on a candidate set (test infrastructure only, numpy fp64).

Sec. 7 step 3 of the paper ("convex sparse solve: compute alpha on the candidates") names the
problem but not an algorithm beyond "Frank-Wolfe or entropic mirror descent with small
iterations and certificates" (Sec. 5.3, App. E; App. F sweeps 2, 4, 6 iterations).  This
module writes out entropic mirror descent for the restriction of Eq. (5.1) to the candidate
set S:

    minimise over the simplex   f_eps(a) = 1/2 |U_S a - q|^2 + eps * sum_i a_i log a_i ,

with U_S the candidates' key rows as columns (d x n), started from the closed form the hot
path uses, a_0 = softmax(U_S^T q / eps) (the same problem with its quadratic term linearised).

One iteration is the Bregman proximal-gradient step with the negative entropy as the mirror
map, the entropy term of the objective handled exactly:

    g_t   = U_S^T (U_S a_t - q)                       gradient of the quadratic part
    a_t+1 = argmin_a  <g_t, a> + eps * Omega(a) + KL(a || a_t) / eta
          => log a_t+1 = (log a_t - eta * g_t) / (1 + eta * eps) + const,

with eta = 1 / L,  L = max_i |u_i|^2.  L is the smoothness constant of the quadratic part
relative to the entropy: for any direction v and any a in the simplex,
|U v|^2 <= L (sum_i |v_i|)^2 <= L * sum_i v_i^2 / a_i  (Cauchy-Schwarz), so f_eps never increases
along the iterates.  The paper fixes neither the step nor the start: both are this library's reading.

The certificate reported with the result is the Frank-Wolfe duality gap of App. E for the
unregularised problem on the candidate simplex,
    g = <grad f(a), a> - min_j grad f(a)_j,   f(a) = 1/2 |U_S a - q|^2,
which bounds f(a) - min f from above.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np


@dataclass
class EntropicSolve:
    alpha: np.ndarray        # final weights on the candidates, sum 1
    objective: float         # f_eps(alpha)
    residual2: float         # |U alpha - q|^2
    fw_gap: float            # Frank-Wolfe gap of the unregularised problem at alpha
    step: float              # eta
    trace: List[np.ndarray]  # a_0 .. a_iters


def _normalise_log(loga: np.ndarray) -> np.ndarray:
    loga = loga - loga.max()
    return loga - np.log(np.exp(loga).sum())


def entropic_mirror_descent(U: np.ndarray, q: np.ndarray, eps: float, iters: int) -> EntropicSolve:
    """`iters` mirror-descent steps from a_0 = softmax(U^T q / eps).  U: d x n, columns = candidates."""
    U = np.asarray(U, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    n = U.shape[1]
    assert n >= 1 and eps > 0 and iters >= 0
    s = U.T @ q                                   # candidate scores <u_i, q>
    L = float(np.max(np.sum(U * U, axis=0)))
    eta = 1.0 / L if L > 0 else 0.0
    loga = _normalise_log(s / eps)
    trace = [np.exp(loga)]
    for _ in range(iters):
        a = np.exp(loga)
        y = U @ a                                 # current readout in key space
        g = U.T @ y - s                           # gradient of 1/2 |U a - q|^2
        loga = _normalise_log((loga - eta * g) / (1.0 + eta * eps))
        trace.append(np.exp(loga))
    a = np.exp(loga)
    y = U @ a
    g = U.T @ y - s
    r = y - q
    ent = float(np.sum(a * loga))
    return EntropicSolve(alpha=a, objective=0.5 * float(r @ r) + eps * ent, residual2=float(r @ r),
                         fw_gap=float(g @ a - g.min()), step=eta, trace=trace)


@dataclass
class SparseEntropicResult:
    out: np.ndarray          # fp64 [B, Hq, d]  sum_i alpha_i v_i over the candidates
    alpha: np.ndarray        # fp64 [B, Hq, K_c] weights in the candidates' selection order, 0 padded
    objective: np.ndarray    # fp64 [B, Hq]
    residual2: np.ndarray
    fw_gap: np.ndarray
    step: np.ndarray
    base: object             # the closed-form pass (candidates, gap diagnostics, fallback flags)


def sparse_entropic(geo, q, k_cache, v_cache, block_table, seq_lens, routed_pages, K_c: int, epsilon: float,
                    gap_threshold: float, iters: int) -> SparseEntropicResult:
    """Sec. 7 steps 2-4 with step 3 done by `iters` mirror-descent iterations: the candidate set and
    every diagnostic of the closed-form pass come from `oracle.sparse`; the weights on that set are
    re-solved here and the values are read out with them.  Native cache layout only."""
    import oracle

    base = oracle.sparse(geo, q, k_cache, v_cache, block_table, seq_lens, routed_pages, K_c, epsilon, gap_threshold)
    B, H, d, G = geo.batch, geo.n_q_heads, geo.head_dim, geo.n_q_heads // geo.n_kv_heads
    ps = geo.page_size
    Kf = oracle.bf16_to_f32(np.asarray(k_cache)).astype(np.float64)
    Vf = oracle.bf16_to_f32(np.asarray(v_cache)).astype(np.float64)
    qf = oracle.bf16_to_f32(np.asarray(q)).astype(np.float64)
    assert Kf.ndim == 4 and Kf.shape[1:] == (geo.n_kv_heads, ps, d), "native [pool][kv_head][page][d] layout"
    bt = np.asarray(block_table)
    res = SparseEntropicResult(out=np.zeros((B, H, d)), alpha=np.zeros((B, H, K_c)), objective=np.zeros((B, H)),
                               residual2=np.zeros((B, H)), fw_gap=np.zeros((B, H)), step=np.zeros((B, H)), base=base)
    for b in range(B):
        for h in range(H):
            n = int(base.n_candidates[b, h])
            if n == 0:
                continue
            pos = base.cand_pos[b, h, :n]
            phys = bt[b, pos // ps]
            rows_k = Kf[phys, h // G, pos % ps]          # n x d
            rows_v = Vf[phys, h // G, pos % ps]
            sol = entropic_mirror_descent(rows_k.T, qf[b, h], float(epsilon), iters)
            res.out[b, h] = sol.alpha @ rows_v
            res.alpha[b, h, :n] = sol.alpha
            res.objective[b, h], res.residual2[b, h] = sol.objective, sol.residual2
            res.fw_gap[b, h], res.step[b, h] = sol.fw_gap, sol.step
    return res


@dataclass
class SparseFrankWolfeResult:
    out: np.ndarray          # fp64 [B, Hq, d]  sum_i alpha_i v_i
    fw: object               # oracle.FrankWolfeResult (weights in the candidates' selection order)
    base: object             # the closed-form pass (candidates, gap diagnostics, fallback flags)


def sparse_frank_wolfe(geo, q, k_cache, v_cache, block_table, seq_lens, routed_pages, K_c: int, epsilon: float,
                       gap_threshold: float, iters: int) -> SparseFrankWolfeResult:
    """Sec. 7 steps 2-4 with step 3 done by `iters` Frank-Wolfe iterations on the unregularised problem
    (App. E).  The weights come from the C oracle's mirrored-fp32 Frank-Wolfe (the vertex choices are
    integers); the values are read out with them in fp64.  Native cache layout only."""
    import oracle

    base = oracle.sparse(geo, q, k_cache, v_cache, block_table, seq_lens, routed_pages, K_c, epsilon, gap_threshold)
    fw = oracle.frank_wolfe(geo, q, k_cache, block_table, base.cand_pos, iters)
    B, H, d, G = geo.batch, geo.n_q_heads, geo.head_dim, geo.n_q_heads // geo.n_kv_heads
    ps = geo.page_size
    Vf = oracle.bf16_to_f32(np.asarray(v_cache)).astype(np.float64)
    bt = np.asarray(block_table)
    out = np.zeros((B, H, d))
    for b in range(B):
        for h in range(H):
            n = int(base.n_candidates[b, h])
            if n == 0:
                continue
            pos = base.cand_pos[b, h, :n]
            rows_v = Vf[bt[b, pos // ps], h // G, pos % ps]
            out[b, h] = fw.alpha[b, h, :n].astype(np.float64) @ rows_v
    return SparseFrankWolfeResult(out=out, fw=fw, base=base)
