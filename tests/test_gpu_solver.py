"""GPU parity of the iterative entropic solve (vsa_sparse_decode_entropic / vsa_decode_step_entropic)
against oracle/solver.py on the same seeded bytes.  The candidate set and every discrete diagnostic
must be those of the closed-form pass, bit for bit; the outputs of the iterations are floating
point: `out` within 1e-2 max-abs / 5e-3 relative L2, the certificate and the objective within the
tolerances derived below."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import solver
from paper_2602_13804_b200 import binding as B
from gpu_runner import check_out, lse_tol
from util import geometry, host_arrays
from workloads import WorkloadSpec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def spec(**kw):
    base = dict(name="t", config=9, batch=3, n_q_heads=8, n_kv_heads=2, P=6, K_c=40,
                seq_lens=(700, 333, 90), needles=3, needle_positions="uniform")
    base.update(kw)
    return WorkloadSpec(**base)


def run_entropic(w, iters, fused=False):
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    units = shape.batch * shape.n_q_heads
    P, K_c = w.spec.P, w.spec.K_c
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    out = torch.full((shape.batch, shape.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag, sol = B.alloc_diag(units, DEV), B.alloc_solve(units, DEV)
    sol.fill_(float("nan"))
    flist = torch.full((units,), -1, dtype=torch.int32, device=DEV)
    fcount = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    routed = torch.full((shape.batch, shape.n_q_heads, P), -7, dtype=torch.int32, device=DEV)
    if fused:
        ws = B.alloc_workspace(shape, P, K_c, B.VSA_WS_STEP, DEV)
        B.vsa_decode_step_entropic(shape, wd.q, summ, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, P, K_c,
                                   w.epsilon, w.gap_threshold, iters, out, diag, sol, routed, flist, fcount, ws)
    else:
        ws = B.alloc_workspace(shape, P, K_c, B.VSA_WS_ROUTE, DEV)
        B.vsa_route_pages(shape, wd.q, summ, wd.block_table, wd.seq_lens, P, routed, None, ws)
        B.vsa_sparse_decode_entropic(shape, wd.q, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, routed, P, K_c,
                                     w.epsilon, w.gap_threshold, iters, out, diag, sol, flist, fcount)
    torch.cuda.synchronize()
    n = int(fcount.item())
    return dict(out=out.cpu().numpy(), diag={k: v.numpy() for k, v in B.diag_to_dict(diag).items()},
                solve=sol.cpu().numpy().astype(np.float64), routed=routed.cpu().numpy(),
                fallback=np.sort(flist[:n].cpu().numpy()))


def oracle_entropic(w, iters):
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    rt = oracle.route(geo, q, summ, bt, sl, w.spec.P)
    return rt, solver.sparse_entropic(geo, q, K, V, bt, sl, rt.pages, w.spec.K_c, w.epsilon, w.gap_threshold, iters)


def compare_entropic(w, g, iters):
    rt, o = oracle_entropic(w, iters)
    Bn, H = o.out.shape[:2]
    assert np.array_equal(g["routed"], rt.pages)
    check_out(g["out"], o.out, f"entropic out, {iters} iterations")
    d, base = g["diag"], o.base
    for name, want in (("delta", base.delta), ("delta12", base.delta12), ("s_max", base.s_max)):
        assert np.array_equal(d[name].reshape(Bn, H), want), name
    assert np.array_equal(d["n_candidates"].reshape(Bn, H), base.n_candidates)
    assert np.array_equal(d["fallback"].reshape(Bn, H), base.fallback)
    assert np.array_equal(g["fallback"], np.nonzero(base.fallback.reshape(-1))[0])
    fin = np.isfinite(base.lse)
    assert np.all(np.abs(d["lse"].reshape(Bn, H)[fin] - base.lse[fin]) <= lse_tol(w.epsilon) + 2e-6 * np.abs(base.lse[fin]))
    # Solve record.  Every entry is a sum of a few hundred fp32 terms of size up to S = |k|(|q| + |y|)
    # (several hundred here): an absolute error of some 1e-4 * S / 100, far inside 1e-2 + 1e-3 relative.
    fw, obj, r2, step = (g["solve"][:, i].reshape(Bn, H) for i in range(4))
    has = base.n_candidates > 0
    assert np.all(np.abs(step - o.step)[has] <= 1e-5 * o.step[has])
    for got, want, what in ((fw, o.fw_gap, "fw_gap"), (obj, o.objective, "objective"), (r2, o.residual2, "residual2")):
        err = np.abs(got - want)[has]
        assert np.all(err <= 1e-2 + 1e-3 * np.abs(want[has])), f"{what}: {err.max():.3e}"
    assert np.all(g["solve"].reshape(Bn, H, 4)[~has] == 0.0)
    return o


@pytest.mark.parametrize("iters", [0, 2, 6])
def test_entropic_sparse_pass_matches_the_oracle(iters):
    w = make_workload(spec(), seed=300 + iters)
    o = compare_entropic(w, run_entropic(w, iters), iters)
    if iters:
        assert np.max(np.abs(o.out - o.base.out)) > 1e-4    # the iterations do change the readout


def test_entropic_zero_iterations_equals_the_closed_form_pass():
    w = make_workload(spec(seq_lens=(500, 260, 33)), seed=310)
    g = run_entropic(w, 0)
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    out = torch.zeros((3, 8, 128), dtype=torch.float32, device=DEV)
    diag = B.alloc_diag(24, DEV)
    fl, fc = torch.zeros(24, dtype=torch.int32, device=DEV), torch.zeros(1, dtype=torch.int32, device=DEV)
    B.vsa_sparse_decode(shape, wd.q, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens,
                        torch.from_numpy(g["routed"]).to(DEV), 6, 40, w.epsilon, w.gap_threshold, out, diag, fl, fc)
    torch.cuda.synchronize()
    assert np.max(np.abs(out.cpu().numpy() - g["out"])) < 2e-5
    d0 = {k: v.numpy() for k, v in B.diag_to_dict(diag).items()}
    for name in ("delta", "delta12", "s_max", "n_candidates", "fallback", "leak_bound"):
        assert np.array_equal(d0[name], g["diag"][name])
    assert np.max(np.abs(d0["lse"] - g["diag"]["lse"])) < 1e-4


def test_entropic_fused_step_equals_separate_calls_and_falls_back_to_dense():
    w = make_workload(spec(needles=0), seed=311)      # needle-free heads: small gaps, units fall back
    a, b = run_entropic(w, 4), run_entropic(w, 4, fused=True)
    assert np.array_equal(a["routed"], b["routed"]) and np.array_equal(a["fallback"], b["fallback"])
    assert np.array_equal(a["solve"], b["solve"])
    flagged = a["fallback"]
    assert len(flagged) > 0
    keep = np.ones(24, bool)
    keep[flagged] = False
    assert np.array_equal(a["out"].reshape(24, -1)[keep], b["out"].reshape(24, -1)[keep])
    # flagged units: the fused step has run the dense pass over them
    q, K, V, bt, sl = host_arrays(w)
    mask = np.zeros(24, np.int32)
    mask[flagged] = 1
    dn = oracle.dense(geometry(w), q, K, V, bt, sl, w.epsilon, unit_mask=mask.reshape(3, 8))
    check_out(b["out"].reshape(24, -1)[flagged], dn.out.reshape(24, -1)[flagged], "dense rows of the entropic step")


def test_entropic_full_candidate_tile_and_degenerate_sets():
    # K_c = 256 with every slot filled (the largest tile), and a second sequence of one token
    # (one candidate: weight 1, zero gap, objective = 1/2 |k - q|^2 exactly)
    w = make_workload(spec(batch=2, seq_lens=(9000, 1), P=32, K_c=256, needles=6), seed=312)
    g = run_entropic(w, 6)
    o = compare_entropic(w, g, 6)
    assert o.base.n_candidates[0].min() == 256 and o.base.n_candidates[1].max() == 1
    fw = g["solve"][:, 0].reshape(2, 8)
    assert np.all(np.abs(fw[1]) < 1e-3)
    # more units than SMs (the shape every batch of the benchmark uses)
    w = make_workload(spec(batch=24, seq_lens=(400,) * 24, P=8, K_c=100, needles=2), seed=313)
    w.gap_threshold = -math.inf                         # no unit is handed to the dense pass
    compare_entropic(w, run_entropic(w, 2, fused=True), 2)


def test_entropic_objective_does_not_increase_with_iterations():
    w = make_workload(spec(), seed=314)
    prev = None
    for iters in (0, 1, 2, 4, 8):
        obj = run_entropic(w, iters)["solve"][:, 1]
        if prev is not None:
            assert np.all(obj <= prev + 1e-3 + 1e-5 * np.abs(prev))
        prev = obj


# ------------------------------------------------------------------------------------- Frank-Wolfe

def run_fw(w, iters, fused=False):
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    units = shape.batch * shape.n_q_heads
    P, K_c = w.spec.P, w.spec.K_c
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    out = torch.full((shape.batch, shape.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag, sol = B.alloc_diag(units, DEV), B.alloc_solve(units, DEV)
    sol.fill_(float("nan"))
    flist = torch.full((units,), -1, dtype=torch.int32, device=DEV)
    fcount = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    routed = torch.full((shape.batch, shape.n_q_heads, P), -7, dtype=torch.int32, device=DEV)
    if fused:
        ws = B.alloc_workspace(shape, P, K_c, B.VSA_WS_STEP, DEV)
        B.vsa_decode_step_frank_wolfe(shape, wd.q, summ, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, P, K_c,
                                      w.epsilon, w.gap_threshold, iters, out, diag, sol, routed, flist, fcount, ws)
    else:
        ws = B.alloc_workspace(shape, P, K_c, B.VSA_WS_ROUTE, DEV)
        B.vsa_route_pages(shape, wd.q, summ, wd.block_table, wd.seq_lens, P, routed, None, ws)
        B.vsa_sparse_decode_frank_wolfe(shape, wd.q, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, routed, P,
                                        K_c, w.epsilon, w.gap_threshold, iters, out, diag, sol, flist, fcount)
    torch.cuda.synchronize()
    n = int(fcount.item())
    return dict(out=out.cpu().numpy(), diag={k: v.numpy() for k, v in B.diag_to_dict(diag).items()},
                solve=sol.cpu().numpy(), routed=routed.cpu().numpy(), fallback=np.sort(flist[:n].cpu().numpy()))


def compare_fw(w, g, iters):
    """The vertex choices are integers: the solve record (every field a product of the mirrored fp32
    arithmetic) must match the oracle bit for bit; `out` is an fp32 gather compared with a tolerance."""
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    rt = oracle.route(geo, q, summ, bt, sl, w.spec.P)
    o = solver.sparse_frank_wolfe(geo, q, K, V, bt, sl, rt.pages, w.spec.K_c, w.epsilon, w.gap_threshold, iters)
    Bn, H = o.out.shape[:2]
    assert np.array_equal(g["routed"], rt.pages)
    got = g["solve"].reshape(Bn, H, 4)
    for i, (name, want) in enumerate((("fw_gap", o.fw.fw_gap), ("objective", o.fw.objective),
                                      ("residual2", o.fw.residual2), ("step", o.fw.step))):
        assert np.array_equal(got[:, :, i].view(np.uint32), want.view(np.uint32)), f"{name} differs"
    check_out(g["out"], o.out, f"frank-wolfe out, {iters} iterations")
    d, base = g["diag"], o.base
    for name, want in (("delta", base.delta), ("delta12", base.delta12), ("s_max", base.s_max)):
        assert np.array_equal(d[name].reshape(Bn, H), want), name
    assert np.array_equal(d["n_candidates"].reshape(Bn, H), base.n_candidates)
    assert np.array_equal(d["fallback"].reshape(Bn, H), base.fallback)
    fin = np.isfinite(base.lse)
    assert np.all(np.abs(d["lse"].reshape(Bn, H)[fin] - base.lse[fin]) <= lse_tol(w.epsilon) + 2e-6 * np.abs(base.lse[fin]))
    return o


@pytest.mark.parametrize("iters", [0, 1, 3, 6])
def test_frank_wolfe_pass_matches_the_oracle(iters):
    w = make_workload(spec(), seed=320 + iters)
    o = compare_fw(w, run_fw(w, iters), iters)
    assert np.all(np.count_nonzero(o.fw.alpha, axis=-1) <= iters + 1)


def test_frank_wolfe_needle_free_heads_and_the_fused_step():
    # flat heads: many near-equal gradient entries, the case where an unmirrored argmin would drift
    w = make_workload(spec(needles=0, seq_lens=(500, 260, 33)), seed=330)
    w.gap_threshold = -math.inf
    compare_fw(w, run_fw(w, 6), 6)
    compare_fw(w, run_fw(w, 6, fused=True), 6)


def test_frank_wolfe_full_tile_and_single_candidate():
    w = make_workload(spec(batch=2, seq_lens=(9000, 1), P=32, K_c=256, needles=6), seed=331)
    w.gap_threshold = -math.inf
    g = run_fw(w, 6, fused=True)
    o = compare_fw(w, g, 6)
    assert o.base.n_candidates[0].min() == 256 and o.base.n_candidates[1].max() == 1
    assert np.all(g["solve"].reshape(2, 8, 4)[1, :, 3] == 0.0)      # one candidate: no step to take


def test_frank_wolfe_duplicate_keys_tie_to_the_lower_position():
    w = make_workload(spec(batch=1, n_q_heads=4, n_kv_heads=2, seq_lens=(64,), P=4, K_c=64, needles=0), seed=332)
    k = w.k_cache.clone()
    p0, p1 = int(w.block_table[0, 0]), int(w.block_table[0, 2])
    k[p1] = k[p0]                                  # tokens 32..47 repeat tokens 0..15, both kv heads
    w.k_cache = k
    w.gap_threshold = -math.inf
    compare_fw(w, run_fw(w, 5), 5)


@pytest.mark.parametrize("kind", ["eg", "fw"])
def test_solvers_with_a_single_candidate_per_unit(kind):
    # K_c = 1: the candidate set is the best token alone; weight 1, zero gap, no step
    w = make_workload(spec(K_c=1, P=2, seq_lens=(200, 90, 40)), seed=340)
    w.gap_threshold = -math.inf
    g = run_entropic(w, 3) if kind == "eg" else run_fw(w, 3)
    if kind == "eg":
        compare_entropic(w, g, 3)
    else:
        compare_fw(w, g, 3)
    sol = np.asarray(g["solve"], dtype=np.float64).reshape(24, 4)
    assert np.all(np.abs(sol[:, 0]) < 1e-3)
