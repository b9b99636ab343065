"""GPU parity of the two-level page routing (representative per 16 pages, exact scores inside the kept
super-pages) against the oracle: representatives and chosen pages bit-exact, kept super-pages, routed pages
and scores bit-exact, and the step built on it equal to the oracle's step on the same routed pages."""
import numpy as np
import pytest
import torch

import oracle
from gpu_runner import check_out, lse_tol
from paper_2602_13804_b200 import binding as B
from util import bits, geometry, host_arrays
from workloads import WorkloadSpec, config_spec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(w, P_super, P, K_c):
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    units = shape.batch * shape.n_q_heads
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    ns = B.n_super_pages(shape)
    sup = torch.full((shape.batch, ns, shape.n_kv_heads, 128), 7.0, dtype=torch.bfloat16, device=DEV)
    rep = torch.full((shape.batch, ns, shape.n_kv_heads), -9, dtype=torch.int32, device=DEV)
    B.vsa_build_super_summaries(shape, summ, wd.block_table, wd.seq_lens, None, sup, rep)
    routed = torch.full((shape.batch, shape.n_q_heads, P), -7, dtype=torch.int32, device=DEV)
    rscores = torch.zeros((shape.batch, shape.n_q_heads, P), dtype=torch.float32, device=DEV)
    srouted = torch.full((shape.batch, shape.n_q_heads, P_super), -7, dtype=torch.int32, device=DEV)
    ws = B.alloc_workspace(shape, P_super, 0, B.VSA_WS_ROUTE_TWO_LEVEL, DEV)
    for _ in range(2):     # twice: nothing of the first call may leak into the second
        B.vsa_route_pages_two_level(shape, wd.q, summ, sup, wd.block_table, wd.seq_lens, P_super, P, routed, rscores,
                                    srouted, ws)
    out = torch.full((shape.batch, shape.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag = B.alloc_diag(units, DEV)
    routed2 = torch.full_like(routed, -7)
    flist = torch.full((units,), -1, dtype=torch.int32, device=DEV)
    fcount = torch.full((1,), 55, dtype=torch.int32, device=DEV)
    ws2 = B.alloc_workspace(shape, P_super, K_c, B.VSA_WS_STEP_TWO_LEVEL, DEV)
    B.vsa_decode_step_two_level(shape, wd.q, summ, sup, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, P_super,
                                P, K_c, w.epsilon, w.gap_threshold, out, diag, routed2, flist, fcount, ws2)
    torch.cuda.synchronize()
    return dict(sup=bits(sup), rep=rep.cpu().numpy(), routed=routed.cpu().numpy(), rscores=rscores.cpu().numpy(),
                srouted=srouted.cpu().numpy(), out=out.cpu().numpy(), diag=B.diag_to_dict(diag),
                routed2=routed2.cpu().numpy(), fb=np.sort(flist[: int(fcount.item())].cpu().numpy()))


def _compare(w, g, P_super, P, K_c):
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    sup, rep = oracle.build_super_summaries(geo, summ, bt, sl)
    assert np.array_equal(g["rep"], rep), "chosen pages differ"
    assert np.array_equal(g["sup"], sup), "representatives differ"
    tl = oracle.route_two_level(geo, q, summ, sup, bt, sl, P_super, P)
    assert np.array_equal(g["srouted"], tl.supers), "kept super-pages differ"
    assert np.array_equal(g["routed"], tl.pages) and np.array_equal(g["rscores"], tl.scores)
    assert np.array_equal(g["routed2"], tl.pages), "routed pages of the step differ"
    sp = oracle.sparse(geo, q, K, V, bt, sl, tl.pages, K_c, w.epsilon, w.gap_threshold)
    Bn, H = geo.batch, geo.n_q_heads
    d = {k: v.numpy().reshape(Bn, H) for k, v in g["diag"].items()}
    assert np.array_equal(d["delta"], sp.delta) and np.array_equal(d["n_candidates"], sp.n_candidates)
    assert np.array_equal(d["fallback"], sp.fallback)
    flagged = np.nonzero(sp.fallback.reshape(-1))[0]
    assert np.array_equal(g["fb"], flagged)
    want = sp.out.copy()
    if len(flagged):
        dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon, unit_mask=sp.fallback)
        want[sp.fallback.astype(bool)] = dn.out[sp.fallback.astype(bool)]
    check_out(g["out"], want, "two-level step out")
    # how much of the exact routing survives the pre-filter (reported, asserted where the test says so)
    exact = oracle.route(geo, q, summ, bt, sl, P)
    hit = tot = 0
    for b in range(Bn):
        for h in range(H):
            e = set(int(x) for x in exact.pages[b, h] if x >= 0)
            hit += len(e & set(int(x) for x in tl.pages[b, h]))
            tot += len(e)
    return hit / tot


@pytest.mark.parametrize("P_super", [1, 3, 8])
def test_small_ragged(P_super):
    spec = WorkloadSpec(name="tl", config=9, batch=3, n_q_heads=8, n_kv_heads=2, P=6, K_c=40,
                        seq_lens=(1200, 613, 40), needles=3)
    w = make_workload(spec, seed=911)
    _compare(w, _run(w, P_super, 6, 40), P_super, 6, 40)


def test_fewer_scored_pages_than_P_routes_only_the_scored_ones():
    """One kept super-page holds at most 16 pages: with P = 64 the routed list is those pages and -1
    padding, never a page that was not scored."""
    spec = WorkloadSpec(name="tl", config=9, batch=3, n_q_heads=4, n_kv_heads=4, P=64, K_c=1,
                        seq_lens=(900, 16, 2000), needles=1)
    w = make_workload(spec, seed=915)
    g = _run(w, 1, 64, 1)
    _compare(w, g, 1, 64, 1)
    assert (g["routed"] >= 0).sum(axis=-1).max() <= 16


def test_every_super_page_kept_equals_the_full_scan():
    spec = WorkloadSpec(name="tl", config=9, batch=2, n_q_heads=4, n_kv_heads=2, P=6, K_c=40,
                        seq_lens=(1500, 333), needles=3)
    w = make_workload(spec, seed=912)
    recall = _compare(w, _run(w, 8, 6, 40), 8, 6, 40)
    assert recall == 1.0


def test_identical_pages_tie_to_the_lowest_page_and_super_page():
    spec = WorkloadSpec(name="tl", config=9, batch=1, n_q_heads=4, n_kv_heads=2, P=5, K_c=32, seq_lens=(2048,),
                        needles=0)
    w = make_workload(spec, seed=913)
    first = int(w.block_table[0, 0])
    for l in range(1, 128):
        w.k_cache[int(w.block_table[0, l])] = w.k_cache[first]
    _compare(w, _run(w, 2, 5, 32), 2, 5, 32)


def test_gqa8_and_a_long_sequence_recall():
    spec = config_spec(2, batch=2, T=32768, n_q_heads=16, n_kv_heads=2)
    w = make_workload(spec, seed=914)
    recall = _compare(w, _run(w, 32, 32, 256), 32, 32, 256)
    assert recall >= 0.9, recall
