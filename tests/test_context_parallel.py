"""Context-parallel (sequence-sharded) variant on CPU: gloo ranks, each holding a contiguous range of
every sequence's pages.  The per-rank results come from the oracle on the rank's shard; the exchanges
under test are paper_2602_13804_b200.context_parallel.  What must hold: the merged top-P pages and their
scores, the merged candidate set and the gap are IDENTICAL to the single-process oracle's; the combined
readouts (sparse and dense) agree with it to 1e-12."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from util import bits
from workloads import WorkloadSpec, make_workload

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
P, K_C = 6, 20


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spec():
    return WorkloadSpec(name="cp", config=7, batch=2, n_q_heads=4, n_kv_heads=2, P=P, K_c=K_C,
                        seq_lens=(700, 333), needles=3)


def _geo(w, batch=None, hq=None, hkv=None, max_pages=None):
    return oracle.Geometry(batch=batch or 2, n_q_heads=hq or 4, n_kv_heads=hkv or 2,
                           max_pages_per_seq=max_pages or w.max_pages_per_seq, num_pool_pages=w.pool_pages)


def _rank_main(rank, world, port):
    sys.path.insert(0, ROOT)
    from paper_2602_13804_b200 import context_parallel as cp
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = make_workload(_spec(), seed=707)
        q, K, V = bits(w.q), bits(w.k_cache), bits(w.v_cache)
        bt, sl = w.block_table.numpy().astype(np.int32), w.seq_lens.numpy().astype(np.int32)
        B, Hq, G = 2, 4, 2
        eps, tau = w.epsilon, w.gap_threshold

        # ---- the single-process result every rank must reproduce ----
        geo = _geo(w)
        summ = oracle.build_summaries(geo, K, bt, sl)
        full_r = oracle.route(geo, q, summ, bt, sl, P)
        full_s = oracle.sparse(geo, q, K, V, bt, sl, full_r.pages, K_C, eps, tau)
        full_d = oracle.dense(geo, q, K, V, bt, sl, eps)

        # ---- this rank's shard: pages [lo, hi) of every sequence ----
        n_pages = (sl + 15) // 16
        lo = np.array([cp.page_range(int(n), rank, world)[0] for n in n_pages])
        hi = np.array([cp.page_range(int(n), rank, world)[1] for n in n_pages])
        assert np.all(hi > lo)
        mp_ = int((hi - lo).max())
        bt_s = np.full((B, mp_), -1, np.int32)
        sl_s = np.zeros(B, np.int32)
        for b in range(B):
            bt_s[b, : hi[b] - lo[b]] = bt[b, lo[b]:hi[b]]
            sl_s[b] = min(int(sl[b]), hi[b] * 16) - lo[b] * 16
        geo_s = _geo(w, max_pages=mp_)

        # 1. page routing: local top-P -> merged global top-P
        loc = oracle.route(geo_s, q, summ, bt_s, sl_s, P)
        glob_pages = np.where(loc.pages >= 0, loc.pages + lo[:, None, None], -1)
        ms, mi = cp.merge_top(torch.from_numpy(loc.scores), torch.from_numpy(glob_pages), P)
        assert np.array_equal(mi.numpy(), full_r.pages.astype(np.int64)), "merged page set differs"
        assert np.array_equal(ms.numpy(), full_r.scores), "merged page scores differ"

        # 2. token routing on the routed pages this rank owns: local top-(K_c + 1) -> merged candidates
        routed = mi.numpy()
        mine = np.full((B, Hq, P), -1, np.int32)
        for b in range(B):
            for h in range(Hq):
                own = [p - lo[b] for p in routed[b, h] if lo[b] <= p < hi[b]]
                mine[b, h, : len(own)] = own
        ls = oracle.sparse(geo_s, q, K, V, bt_s, sl_s, mine, K_C + 1, eps, tau)
        sc = np.full((B, Hq, K_C + 1), -np.inf, np.float32)
        gpos = np.full((B, Hq, K_C + 1), -1, np.int64)
        for b in range(B):
            for h in range(Hq):
                for j, p in enumerate(ls.cand_pos[b, h]):
                    if p < 0:
                        continue
                    page, t = bt_s[b, p // 16], p % 16
                    sc[b, h, j] = oracle.canon_dot(q[b, h], K[page, h // G, t])
                    gpos[b, h, j] = lo[b] * 16 + p
        ts, ti = cp.merge_top(torch.from_numpy(sc), torch.from_numpy(gpos), K_C + 1)
        cand, delta = cp.gap_from_merged(ts, ti, K_C)
        for b in range(B):
            for h in range(Hq):
                want = set(int(x) for x in full_s.cand_pos[b, h] if x >= 0)
                got = set(int(x) for x in cand[b, h].tolist() if x >= 0)
                assert got == want, "merged candidate set differs"
        assert np.array_equal(delta.numpy(), full_s.delta), "gap statistic differs"

        # 3. readout over this rank's members of the candidate set, then the combine.  The partial readout
        # is the oracle's dense attention on a cache that holds exactly those tokens (one tiny "sequence"
        # per unit), so no formula of the method is retyped here.
        units = B * Hq
        rows = K_C + 1
        mini_pages = (rows + 15) // 16
        Kp = np.zeros((units * mini_pages, 1, 16, 128), np.uint16)
        Vp = np.zeros_like(Kp)
        bt_m = np.arange(units * mini_pages, dtype=np.int32).reshape(units, mini_pages)
        sl_m = np.ones(units, np.int32)
        empty = np.zeros(units, bool)
        for b in range(B):
            for h in range(Hq):
                u = b * Hq + h
                members = [int(p) for p in cand[b, h].tolist() if p >= 0 and lo[b] * 16 <= p < hi[b] * 16]
                empty[u] = not members
                sl_m[u] = max(1, len(members))
                for j, p in enumerate(members):
                    page = bt[b, p // 16]
                    Kp[u * mini_pages + j // 16, 0, j % 16] = K[page, h // G, p % 16]
                    Vp[u * mini_pages + j // 16, 0, j % 16] = V[page, h // G, p % 16]
        geo_m = oracle.Geometry(batch=units, n_q_heads=1, n_kv_heads=1, max_pages_per_seq=mini_pages,
                                num_pool_pages=units * mini_pages)
        part = oracle.dense(geo_m, q.reshape(units, 1, 128), Kp, Vp, bt_m, sl_m, eps)
        lse_p = np.where(empty, -np.inf, part.lse.reshape(units))
        out_c, lse_c = cp.combine_partials(torch.from_numpy(part.out.reshape(units, 128)), torch.from_numpy(lse_p))
        assert np.max(np.abs(out_c.numpy() - full_s.out.reshape(units, 128))) <= 1e-12
        assert np.max(np.abs(lse_c.numpy() - full_s.lse.reshape(units))) <= 1e-12

        # dense attention of the sharded sequences: per-rank dense over the shard, combined
        dn = oracle.dense(geo_s, q, K, V, bt_s, sl_s, eps)
        out_d, lse_d = cp.combine_partials(torch.from_numpy(dn.out), torch.from_numpy(dn.lse))
        assert np.max(np.abs(out_d.numpy() - full_d.out)) <= 1e-12
        assert np.max(np.abs(lse_d.numpy() - full_d.lse)) <= 1e-12
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_sequence_sharded_ranks_agree_with_one_process(world):
    mp.spawn(_rank_main, args=(world, _free_port()), nprocs=world, join=True)


def test_merge_order_ties_and_signed_zero():
    """The merge alone, one process: equal scores go to the lower index, -0 equals +0, unused slots lose."""
    sys.path.insert(0, ROOT)
    from paper_2602_13804_b200 import context_parallel as cp
    port = _free_port()
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK="0", WORLD_SIZE="1")
    dist.init_process_group("gloo", rank=0, world_size=1)
    try:
        s = torch.tensor([[1.0, -0.0, 0.0, 1.0, 5.0, 9.0]])
        i = torch.tensor([[7, 3, 2, 4, -1, 1]])
        ms, mi = cp.merge_top(s, i, 5)
        assert mi.tolist() == [[1, 4, 7, 2, 3]] and ms.tolist() == [[9.0, 1.0, 1.0, 0.0, 0.0]]
        ms, mi = cp.merge_top(s[:, :2], i[:, :2], 4)
        assert mi.tolist() == [[7, 3, -1, -1]]
        cand, delta = cp.gap_from_merged(torch.tensor([[3.0, 2.0, 0.5]]), torch.tensor([[5, 6, 9]]), 2)
        assert cand.tolist() == [[5, 6]] and delta.tolist() == [2.5]
        cand, delta = cp.gap_from_merged(torch.tensor([[3.0, 2.0, float("-inf")]]), torch.tensor([[5, 6, -1]]), 2)
        assert delta.tolist() == [float("inf")]
    finally:
        dist.destroy_process_group()
