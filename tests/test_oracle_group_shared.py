"""Pins of the oracle's group-shared routing (the heads of a GQA group route as one query: summed page
scores, summed token scores, one page set and one candidate set per KV head; each head's softmax and
diagnostics use its own scores).  The variant is a reading, so the pins are its reductions and properties:
groups of one reproduce the per-head path bit for bit; sums are fp32 in ascending head order; both
selections dominate (brute force); each head's readout equals a library softmax over the shared set;
everything routed and kept reduces to dense attention; the diagnostics from every token's scores."""
import numpy as np
import pytest
import torch

import oracle
from util import bits, gathered_kv, geometry, host_arrays
from workloads import WorkloadSpec, make_workload


def _w(hq=8, hkv=2, seed=950, **kw):
    base = dict(name="gs", config=9, batch=2, n_q_heads=hq, n_kv_heads=hkv, P=5, K_c=30,
                seq_lens=(700, 333), needles=3, needle_positions="uniform")
    base.update(kw)
    return make_workload(WorkloadSpec(**base), seed=seed)


def test_groups_of_one_reduce_to_the_per_head_path_bit_for_bit():
    w = _w(hq=4, hkv=4)
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    a, b = oracle.route(geo, q, summ, bt, sl, 5), oracle.route_group(geo, q, summ, bt, sl, 5)
    assert np.array_equal(a.pages, b.pages) and np.array_equal(a.scores, b.scores)
    sa = oracle.sparse(geo, q, K, V, bt, sl, a.pages, 30, w.epsilon, w.gap_threshold)
    sb = oracle.sparse_group(geo, q, K, V, bt, sl, b.pages, 30, w.epsilon, w.gap_threshold)
    for f in ("out", "delta", "delta12", "s_max", "lse", "leak_bound", "n_candidates", "fallback", "cand_pos"):
        assert np.array_equal(getattr(sa, f), getattr(sb, f)), f


def test_page_scores_are_fp32_sums_in_ascending_head_order_and_the_selection_dominates():
    w = _w()
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    G, P = 4, 5
    per_head = oracle.route(geo, q, summ, bt, sl, 1, want_all_scores=True).all_scores
    r = oracle.route_group(geo, q, summ, bt, sl, P)
    for b in range(geo.batch):
        nb = (int(sl[b]) + 15) // 16
        for g in range(geo.n_kv_heads):
            tot = per_head[b, g * G, :nb].copy()
            for h in range(1, G):
                tot = (tot + per_head[b, g * G + h, :nb]).astype(np.float32)
            order = sorted(range(nb), key=lambda l: (-float(tot[l]), l))[:P]
            assert r.pages[b, g].tolist() == order
            assert np.array_equal(r.scores[b, g], tot[order])


def test_candidates_dominate_and_each_head_is_a_library_softmax_over_the_shared_set():
    w = _w()
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    G, P, K_c = 4, 5, 30
    r = oracle.route_group(geo, q, summ, bt, sl, P)
    sp = oracle.sparse_group(geo, q, K, V, bt, sl, r.pages, K_c, w.epsilon, w.gap_threshold)
    f = oracle.bf16_to_f32
    for b in range(geo.batch):
        T = int(sl[b])
        for g in range(geo.n_kv_heads):
            scored = [l * 16 + t for l in r.pages[b, g] if l >= 0 for t in range(16) if l * 16 + t < T]
            sc = {}
            for pos in scored:
                row = K[bt[b, pos // 16], g, pos % 16]
                per = [oracle.canon_dot(q[b, g * G + h], row) for h in range(G)]
                tot = per[0]
                for v in per[1:]:
                    tot = np.float32(tot + v)
                sc[pos] = (tot, per)
            S = [int(p) for p in sp.cand_pos[b, g] if p >= 0]
            assert len(S) == min(K_c, len(scored)) and len(set(S)) == len(S)
            for a in S:                                    # brute-force dominance on the summed scores
                for o in scored:
                    if o not in S:
                        assert sc[a][0] > sc[o][0] or (sc[a][0] == sc[o][0] and a < o)
            k, v = gathered_kv(w, b, g)
            idx = torch.tensor(S)
            for h in range(G):
                u = g * G + h
                logits = (k[idx] @ torch.from_numpy(f(q[b, u]).astype(np.float64))) / w.epsilon
                want = torch.softmax(logits, 0) @ v[idx]
                assert np.max(np.abs(sp.out[b, u] - want.numpy())) <= 1e-12
                assert abs(sp.lse[b, u] - float(torch.logsumexp(logits, 0))) <= 1e-12
                inside = sorted((sc[p][1][h] for p in S), reverse=True)
                outside = [sc[p][1][h] for p in scored if p not in S]
                assert sp.s_max[b, u] == inside[0] and sp.delta12[b, u] == np.float32(inside[0] - inside[1])
                want_delta = np.float32(inside[0] - max(outside)) if outside else np.inf
                assert sp.delta[b, u] == want_delta
                assert sp.fallback[b, u] == int(want_delta < w.gap_threshold and len(S) < T)
                lb = min(1.0, (T - len(S)) * np.exp(-float(want_delta) / w.epsilon))
                assert abs(sp.leak_bound[b, u] - lb) <= 1e-12 * max(lb, 1e-300)
                assert sp.n_candidates[b, u] == len(S)


def test_everything_routed_and_kept_is_dense_attention():
    w = _w(seq_lens=(200, 77), P=16, K_c=256)
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    r = oracle.route_group(geo, q, summ, bt, sl, 16)
    sp = oracle.sparse_group(geo, q, K, V, bt, sl, r.pages, 256, w.epsilon, w.gap_threshold)
    dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon)
    assert np.max(np.abs(sp.out - dn.out)) <= 1e-13 and np.max(np.abs(sp.lse - dn.lse)) <= 1e-12
    assert np.all(np.isinf(sp.delta)) and not sp.fallback.any()
