"""GPU parity of the per-rank kernels of the sequence-sharded (context-parallel) step: the pages of every
sequence are dealt to R emulated ranks (one process, the ranks' kernels run one after the other on the one
GPU - none waits for another), the proposals are merged with the same functions the collectives use, and
the result must be the single-rank oracle's: routed pages, their scores, the candidate set and the gap
statistic bit for bit, readout and log-sum-exp within the tolerances of gpu_runner."""
import os
import tempfile

import numpy as np
import pytest
import torch

import oracle
from gpu_runner import check_out, lse_tol
from paper_2602_13804_b200 import binding as B
from paper_2602_13804_b200 import context_parallel as cp
from util import geometry, host_arrays
from workloads import WorkloadSpec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def spec(**kw):
    base = dict(name="cp", config=9, batch=3, n_q_heads=8, n_kv_heads=2, P=4, K_c=40,
                seq_lens=(700, 333, 45), needles=3, needle_positions="uniform")
    base.update(kw)
    return WorkloadSpec(**base)


def shard_tables(w, world, interleave=False):
    """block tables of the ranks: contiguous page ranges per sequence, or pages dealt round-robin"""
    bt = w.block_table.cpu()
    ps = w.spec.page_size
    tables = [torch.full_like(bt, -1) for _ in range(world)]
    for b in range(bt.shape[0]):
        nb = -(-int(w.seq_lens[b]) // ps)
        for r in range(world):
            if interleave:
                idx = torch.arange(r, nb, world)
            else:
                lo, hi = cp.page_range(nb, r, world)
                idx = torch.arange(lo, hi)
            tables[r][b, idx] = bt[b, idx]
    return [t.to(DEV) for t in tables]


def run_sharded(w, world, interleave=False):
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    P, K_c = w.spec.P, w.spec.K_c
    tables = shard_tables(w, world, interleave)
    ranks = [cp.RankKernels(shape, P, K_c, DEV) for _ in range(world)]
    summ = []
    for r in range(world):     # every rank summarises the pages it holds
        s = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
        B.vsa_build_page_summaries(shape, wd.k_cache, tables[r], wd.seq_lens, None, s)
        summ.append(s)
    prop = [ranks[r].propose_pages(wd.q, summ[r], tables[r], wd.seq_lens) for r in range(world)]
    rs, routed = cp.merge_lists(torch.cat([p[0] for p in prop], -1), torch.cat([p[1] for p in prop], -1), P)
    prop = [ranks[r].propose_tokens(wd.q, wd.k_cache, tables[r], wd.seq_lens, routed) for r in range(world)]
    ms, mi = cp.merge_lists(torch.cat([p[0] for p in prop], -1), torch.cat([p[1] for p in prop], -1), K_c + 1)
    cand, delta = cp.gap_from_merged(ms, mi, K_c)
    parts = [ranks[r].partial_readout(wd.v_cache, tables[r], wd.seq_lens, cand, ms[..., :K_c], w.epsilon)
             for r in range(world)]
    parts = [(o.clone(), l.clone()) for o, l in parts]
    out, lse = cp.combine_lists(torch.stack([p[0] for p in parts]), torch.stack([p[1] for p in parts]))
    torch.cuda.synchronize()
    return dict(routed=routed.cpu().numpy(), rscores=rs.cpu().numpy(), cand=cand.cpu().numpy(),
                delta=delta.cpu().numpy(), out=out.cpu().numpy(), lse=lse.cpu().numpy(),
                owners=[int((l.cpu() > -np.inf).sum()) for _, l in parts])


def compare(w, g):
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    r = oracle.route(geo, q, summ, bt, sl, w.spec.P)
    assert np.array_equal(g["routed"], r.pages), "routed pages differ"
    assert np.array_equal(g["rscores"], r.scores)
    sp = oracle.sparse(geo, q, K, V, bt, sl, r.pages, w.spec.K_c, w.epsilon, w.gap_threshold)
    for b in range(geo.batch):
        for h in range(geo.n_q_heads):
            want = sorted(int(x) for x in sp.cand_pos[b, h] if x >= 0)
            got = sorted(int(x) for x in g["cand"][b, h] if x >= 0)
            assert got == want, (b, h)
    assert np.array_equal(g["delta"], sp.delta), "gap statistic differs"
    check_out(g["out"], sp.out, "sharded readout")
    fin = np.isfinite(sp.lse)
    assert np.all(np.abs(g["lse"][fin] - sp.lse[fin]) <= lse_tol(w.epsilon) + 2e-6 * np.abs(sp.lse[fin]))


@pytest.mark.parametrize("world", [1, 2, 3, 4])
@pytest.mark.parametrize("interleave", [False, True])
def test_sharded_step_equals_the_single_rank_oracle(world, interleave):
    w = make_workload(spec(), seed=800 + world)
    g = run_sharded(w, world, interleave)
    compare(w, g)
    if world > 1:
        assert sum(1 for n in g["owners"] if n > 0) > 1    # the candidates really are spread over ranks


@pytest.mark.parametrize("hq,hkv,page", [(8, 1, 16), (4, 4, 16), (32, 2, 16), (8, 2, 32)])
def test_group_sizes_and_32_token_pages(hq, hkv, page):
    w = make_workload(spec(n_q_heads=hq, n_kv_heads=hkv, page_size=page, seq_lens=(1500, 700, 33), P=5, K_c=64),
                      seed=820 + hq + page)
    compare(w, run_sharded(w, 3))


def test_ranks_without_pages_short_sequences_and_large_sets():
    # 5 ranks for sequences of 1-3 pages (some ranks hold nothing), K_c larger than the scored tokens, and
    # the largest candidate count
    w = make_workload(spec(batch=4, seq_lens=(40, 7, 16, 33), P=8, K_c=128), seed=830)
    compare(w, run_sharded(w, 5))
    w = make_workload(spec(batch=2, n_q_heads=2, n_kv_heads=1, seq_lens=(5000, 2049), P=128, K_c=700), seed=831)
    compare(w, run_sharded(w, 2, interleave=True))


def test_engineered_ties_across_ranks():
    # byte-identical pages held by different ranks: the merge must keep the lower page / position
    w = make_workload(spec(batch=2, seq_lens=(160, 96), needles=0, P=3, K_c=20), seed=840)
    k = w.k_cache.clone()
    bt = w.block_table
    for dst in (3, 4, 7):
        k[int(bt[0, dst])] = k[int(bt[0, 1])]
    k[int(bt[1, 2])] = k[int(bt[1, 0])]
    w.k_cache = k
    compare(w, run_sharded(w, 2, interleave=True))
    compare(w, run_sharded(w, 4))


def test_driver_with_a_process_group_of_one():
    import torch.distributed as dist
    w = make_workload(spec(), seed=850)
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    store = os.path.join(tempfile.mkdtemp(), "store")
    dist.init_process_group("gloo", init_method=f"file://{store}", rank=0, world_size=1)
    try:
        rank = cp.RankKernels(shape, w.spec.P, w.spec.K_c, DEV)
        out, lse, delta, routed, cand = cp.decode_step(rank, wd.q, summ, wd.k_cache, wd.v_cache, wd.block_table,
                                                       wd.seq_lens, w.epsilon)
        torch.cuda.synchronize()
    finally:
        dist.destroy_process_group()
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    r = oracle.route(geo, q, oracle.build_summaries(geo, K, bt, sl), bt, sl, w.spec.P)
    sp = oracle.sparse(geo, q, K, V, bt, sl, r.pages, w.spec.K_c, w.epsilon, w.gap_threshold)
    assert np.array_equal(routed.cpu().numpy(), r.pages) and np.array_equal(delta.cpu().numpy(), sp.delta)
    check_out(out.cpu().numpy(), sp.out, "driver readout")
