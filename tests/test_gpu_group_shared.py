"""GPU parity of the group-shared step (the heads of a GQA group route as one query) against the oracle:
routed page lists, candidate-derived diagnostics and fallback decisions bit-exact, outputs within the
library's tolerances, flagged units equal to dense attention."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_runner import check_out, lse_tol
from paper_2602_13804_b200 import binding as B
from util import geometry, host_arrays
from workloads import WorkloadSpec, config_spec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_and_compare(w, P=None, K_c=None, tau=None):
    P, K_c = P or w.spec.P, K_c or w.spec.K_c
    tau = w.gap_threshold if tau is None else tau
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    units = shape.batch * shape.n_q_heads
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    out = torch.full((shape.batch, shape.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag = B.alloc_diag(units, DEV)
    routed = torch.full((shape.batch, shape.n_kv_heads, P), -7, dtype=torch.int32, device=DEV)
    flist = torch.full((units,), -1, dtype=torch.int32, device=DEV)
    fcount = torch.full((1,), 31, dtype=torch.int32, device=DEV)
    ws = B.alloc_workspace(shape, P, K_c, B.VSA_WS_STEP, DEV)
    for _ in range(2):
        B.vsa_decode_step_group_shared(shape, wd.q, summ, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, P, K_c,
                                       w.epsilon, tau, out, diag, routed, flist, fcount, ws)
    torch.cuda.synchronize()

    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    o_sum = oracle.build_summaries(geo, K, bt, sl)
    r = oracle.route_group(geo, q, o_sum, bt, sl, P)
    assert np.array_equal(routed.cpu().numpy(), r.pages), "routed pages differ"
    sp = oracle.sparse_group(geo, q, K, V, bt, sl, r.pages, K_c, w.epsilon, tau)
    Bn, H = geo.batch, geo.n_q_heads
    d = {k: v.numpy().reshape(Bn, H) for k, v in B.diag_to_dict(diag).items()}
    for name, want in (("delta", sp.delta), ("delta12", sp.delta12), ("s_max", sp.s_max)):
        assert np.array_equal(d[name], want), f"diag.{name} differs"
    assert np.array_equal(d["n_candidates"], sp.n_candidates) and np.array_equal(d["fallback"], sp.fallback)
    assert not d["status"].any()
    flagged = np.nonzero(sp.fallback.reshape(-1))[0]
    assert np.array_equal(np.sort(flist[: int(fcount.item())].cpu().numpy()), flagged)
    lb = d["leak_bound"].astype(np.float64)
    assert np.all(np.abs(lb - sp.leak_bound) <= 1e-3 * sp.leak_bound + 1e-37)
    want_out, want_lse = sp.out.copy(), sp.lse.copy()
    if len(flagged):
        dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon, unit_mask=sp.fallback)
        m = sp.fallback.astype(bool)
        want_out[m], want_lse[m] = dn.out[m], dn.lse[m]
    check_out(out.cpu().numpy(), want_out, "group-shared out")
    fin = np.isfinite(want_lse)
    assert np.all(np.abs(d["lse"][fin] - want_lse[fin]) <= lse_tol(w.epsilon) + 2e-6 * np.abs(want_lse[fin]))
    return float(len(flagged)) / (Bn * H)


@pytest.mark.parametrize("hq,hkv", [(8, 2), (8, 1), (4, 2), (4, 4)])
@pytest.mark.parametrize("needles", [3, 0])
def test_small_ragged_every_group_size(hq, hkv, needles):
    spec = WorkloadSpec(name="gs", config=9, batch=3, n_q_heads=hq, n_kv_heads=hkv, P=5, K_c=30,
                        seq_lens=(700, 333, 40), needles=needles, needle_positions="uniform")
    _run_and_compare(make_workload(spec, seed=960 + hq + hkv))


def test_thresholds_and_fewer_tokens_than_candidates():
    spec = WorkloadSpec(name="gs", config=9, batch=2, n_q_heads=8, n_kv_heads=2, P=16, K_c=256,
                        seq_lens=(200, 77), needles=2)
    w = make_workload(spec, seed=970)
    assert _run_and_compare(w) == 0.0                      # everything kept: no gap, no fallback
    spec = WorkloadSpec(name="gs", config=9, batch=2, n_q_heads=8, n_kv_heads=2, P=4, K_c=24,
                        seq_lens=(900, 500), needles=2)
    w = make_workload(spec, seed=971)
    assert _run_and_compare(w, tau=math.inf) == 1.0        # every unit to the dense pass
    assert _run_and_compare(w, tau=-math.inf) == 0.0


def test_engineered_ties():
    spec = WorkloadSpec(name="gs", config=9, batch=1, n_q_heads=8, n_kv_heads=2, P=5, K_c=40, seq_lens=(1024,),
                        needles=0)
    w = make_workload(spec, seed=972)
    first = int(w.block_table[0, 0])
    for l in range(1, 64):                                  # identical pages: ties in both selections
        w.k_cache[int(w.block_table[0, l])] = w.k_cache[first]
    _run_and_compare(w)


def test_largest_sizes_and_config1_shape():
    w = make_workload(config_spec(2, batch=2, T=32768, P=128, K_c=2048), seed=973)
    _run_and_compare(w)
    w = make_workload(config_spec(1, batch=2), seed=974)
    _run_and_compare(w)


def test_gqa8_ragged():
    w = make_workload(config_spec(4, batch=6, ragged_T=(300, 9000)), seed=975)
    _run_and_compare(w)
