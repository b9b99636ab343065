"""Runs a workload through the C-ABI library on the GPU and through the oracle on the CPU, and
compares the two.  Used by the GPU parity tests."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

import oracle
from paper_2602_13804_b200 import binding as B
from util import bits, geometry, host_arrays
from workloads import Workload

# tolerances of the floating-point outputs (fp32 accumulation of bf16 inputs vs fp64 oracle)
OUT_MAX_ABS = 1e-2
OUT_REL_L2 = 5e-3


@dataclass
class GpuRun:
    summaries: torch.Tensor
    routed_pages: np.ndarray
    routed_scores: np.ndarray
    out_sparse: np.ndarray      # output of vsa_sparse_decode alone
    diag_sparse: dict
    out: np.ndarray             # after vsa_dense_decode_fallback
    diag: dict
    fallback_units: np.ndarray  # sorted unit ids
    step_out: np.ndarray        # output of the single-call vsa_decode_step
    step_diag: dict
    step_routed: np.ndarray
    step_fallback_units: np.ndarray


def run_gpu(w: Workload, P: Optional[int] = None, K_c: Optional[int] = None, epsilon: Optional[float] = None,
            gap_threshold: Optional[float] = None, device="cuda:0", summaries: Optional[torch.Tensor] = None) -> GpuRun:
    P = P or w.spec.P
    K_c = K_c or w.spec.K_c
    eps = w.epsilon if epsilon is None else epsilon
    tau = w.gap_threshold if gap_threshold is None else gap_threshold
    wd = w if w.q.is_cuda else w.to(device)
    dev = wd.q.device
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    units = shape.batch * shape.n_q_heads

    if summaries is None:
        summaries = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=dev)
        B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summaries)

    routed = torch.full((shape.batch, shape.n_q_heads, P), -7, dtype=torch.int32, device=dev)
    rscores = torch.zeros((shape.batch, shape.n_q_heads, P), dtype=torch.float32, device=dev)
    ws_r = B.alloc_workspace(shape, P, K_c, B.VSA_WS_ROUTE, dev)
    B.vsa_route_pages(shape, wd.q, summaries, wd.block_table, wd.seq_lens, P, routed, rscores, ws_r)

    out = torch.full((shape.batch, shape.n_q_heads, shape.head_dim), float("nan"), dtype=torch.float32, device=dev)
    diag = B.alloc_diag(units, dev)
    flist = torch.full((units,), -1, dtype=torch.int32, device=dev)
    fcount = torch.full((1,), 12345, dtype=torch.int32, device=dev)
    B.vsa_sparse_decode(shape, wd.q, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, routed, P, K_c, eps, tau,
                        out, diag, flist, fcount)
    out_sparse = out.cpu().numpy().copy()
    diag_sparse = {k: v.numpy() for k, v in B.diag_to_dict(diag).items()}

    ws_d = B.alloc_workspace(shape, P, K_c, B.VSA_WS_DENSE, dev)
    B.vsa_dense_decode_fallback(shape, wd.q, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, flist, fcount, eps,
                                out, diag, ws_d)
    n = int(fcount.item())
    fb = np.sort(flist[:n].cpu().numpy())

    # the fused single call, on fresh buffers
    out2 = torch.full_like(out, float("nan"))
    diag2 = B.alloc_diag(units, dev)
    routed2 = torch.full_like(routed, -7)
    flist2 = torch.full_like(flist, -1)
    fcount2 = torch.full_like(fcount, 777)
    ws_s = B.alloc_workspace(shape, P, K_c, B.VSA_WS_STEP, dev)
    B.vsa_decode_step(shape, wd.q, summaries, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, P, K_c, eps, tau,
                      out2, diag2, routed2, flist2, fcount2, ws_s)
    n2 = int(fcount2.item())
    torch.cuda.synchronize(dev)
    return GpuRun(
        summaries=summaries, routed_pages=routed.cpu().numpy(), routed_scores=rscores.cpu().numpy(),
        out_sparse=out_sparse, diag_sparse=diag_sparse, out=out.cpu().numpy(),
        diag={k: v.numpy() for k, v in B.diag_to_dict(diag).items()}, fallback_units=fb,
        step_out=out2.cpu().numpy(), step_diag={k: v.numpy() for k, v in B.diag_to_dict(diag2).items()},
        step_routed=routed2.cpu().numpy(), step_fallback_units=np.sort(flist2[:n2].cpu().numpy()))


def check_out(got: np.ndarray, want: np.ndarray, what: str):
    got = got.astype(np.float64).reshape(want.shape)
    err = np.max(np.abs(got - want))
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    assert err <= OUT_MAX_ABS, f"{what}: max-abs {err:.3e} > {OUT_MAX_ABS}"
    assert rel <= OUT_REL_L2, f"{what}: relative L2 {rel:.3e} > {OUT_REL_L2}"
    return err, rel


def lse_tol(eps: float) -> float:
    # fp32 score error (<= 11 * 2^-24 * sum|q_i k_i|, a few 1e-4 for the largest scores here) enters
    # the log-sum-exp divided by epsilon; 1e-3 covers the fp32 log/exp and accumulation
    return 1e-3 + 4e-4 / eps


def compare(w: Workload, g: GpuRun, P=None, K_c=None, epsilon=None, gap_threshold=None,
            dense_sample: Optional[int] = None, seed: int = 0) -> dict:
    """Full comparison of a GPU run with the oracle on the same bytes.  With dense_sample=n the
    dense fallback output is checked on n flagged units (chosen with `seed`) instead of all."""
    P = P or w.spec.P
    K_c = K_c or w.spec.K_c
    eps = w.epsilon if epsilon is None else epsilon
    tau = w.gap_threshold if gap_threshold is None else gap_threshold
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    Bn, H = geo.batch, geo.n_q_heads

    # S0: summaries, bit exact on every page a sequence owns
    o_sum = oracle.build_summaries(geo, K, bt, sl)
    g_sum = bits(g.summaries)
    owned = np.concatenate([bt[b, : -(-int(sl[b]) // geo.page_size)] for b in range(Bn) if sl[b] > 0])
    assert np.array_equal(g_sum[owned], o_sum[owned]), "page summaries differ"

    # S1: routed pages (ordered lists) and their scores, bit exact
    r = oracle.route(geo, q, o_sum, bt, sl, P)
    assert np.array_equal(g.routed_pages, r.pages), "routed pages differ"
    assert np.array_equal(g.routed_scores, r.scores), "routed scores differ"
    assert np.array_equal(g.step_routed, r.pages), "routed pages of the fused step differ"

    # S2-S4: candidates' output and diagnostics
    sp = oracle.sparse(geo, q, K, V, bt, sl, r.pages, K_c, eps, tau)
    stats = {}
    stats["sparse_err"] = check_out(g.out_sparse, sp.out, "sparse out")
    d = g.diag_sparse
    for name, want in (("delta", sp.delta), ("delta12", sp.delta12), ("s_max", sp.s_max)):
        assert np.array_equal(d[name].reshape(Bn, H), want), f"diag.{name} differs"
    assert np.array_equal(d["n_candidates"].reshape(Bn, H), sp.n_candidates)
    assert np.array_equal(d["fallback"].reshape(Bn, H), sp.fallback), "fallback flags differ"
    assert not d["status"].any()
    fin = np.isfinite(sp.lse)
    assert np.all(np.abs(d["lse"].reshape(Bn, H)[fin] - sp.lse[fin]) <= lse_tol(eps) + 2e-6 * np.abs(sp.lse[fin]))
    lb = d["leak_bound"].reshape(Bn, H).astype(np.float64)
    # relative 1e-3 (fp32 exp of an argument up to ~100), absolute slack in the fp32 subnormal range
    assert np.all(np.abs(lb - sp.leak_bound) <= 1e-3 * sp.leak_bound + 1e-37)
    flagged = np.nonzero(sp.fallback.reshape(-1))[0]
    assert np.array_equal(g.fallback_units, flagged), "fallback list differs"
    assert np.array_equal(g.step_fallback_units, flagged), "fallback list of the fused step differs"
    stats["fallback_fraction"] = float(len(flagged)) / (Bn * H)

    # S5: dense output for flagged units; everything else untouched
    untouched = np.ones(Bn * H, bool)
    untouched[flagged] = False
    assert np.array_equal(g.out.reshape(Bn * H, -1)[untouched], g.out_sparse.reshape(Bn * H, -1)[untouched])
    assert np.array_equal(g.step_out, g.out), "fused step and separate calls disagree"
    for name in ("delta", "delta12", "s_max", "lse", "leak_bound", "n_candidates", "fallback", "status"):
        assert np.array_equal(g.step_diag[name], g.diag[name], equal_nan=True), f"step diag.{name}"
    if len(flagged):
        check = flagged
        if dense_sample is not None and dense_sample < len(flagged):
            check = np.sort(np.random.default_rng(seed).choice(flagged, dense_sample, replace=False))
        mask = np.zeros(Bn * H, np.int32)
        mask[check] = 1
        dn = oracle.dense(geo, q, K, V, bt, sl, eps, unit_mask=mask.reshape(Bn, H))
        stats["dense_err"] = check_out(g.out.reshape(Bn * H, -1)[check], dn.out.reshape(Bn * H, -1)[check], "dense out")
        glse = g.diag["lse"][check].astype(np.float64)
        want = dn.lse.reshape(-1)[check]
        assert np.all(np.abs(glse - want) <= lse_tol(eps) + 2e-6 * np.abs(want))
    return stats
