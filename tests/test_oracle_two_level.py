"""Pins of the oracle's two-level routing (representative summary per 16 pages, P_super super-pages kept,
exact page scores inside them).  The construction is this library's, so the pins are its special cases and
the properties it claims: the representative is the super-page's max-norm member; keeping every super-page
reproduces the exact routing; the result is the exact top-P of the pages inside the kept super-pages; on
workloads with planted needles the exact routing's pages are recalled."""
import numpy as np
import pytest

import oracle
from util import geometry, host_arrays
from workloads import WorkloadSpec, make_workload


def _spec(**kw):
    base = dict(name="tl", config=9, batch=2, n_q_heads=4, n_kv_heads=2, P=6, K_c=40,
                seq_lens=(1200, 613), needles=3)
    base.update(kw)
    return WorkloadSpec(**base)


def _setup(seed=901, **kw):
    w = make_workload(_spec(**kw), seed=seed)
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    sup, rep = oracle.build_super_summaries(geo, summ, bt, sl)
    return w, geo, q, summ, sup, rep, bt, sl


def test_representative_is_the_max_norm_member_of_its_super_page():
    w, geo, q, summ, sup, rep, bt, sl = _setup()
    f = oracle.bf16_to_f32
    for b in range(geo.batch):
        nb = (int(sl[b]) + 15) // 16
        for s in range(rep.shape[1]):
            for g in range(geo.n_kv_heads):
                pages = list(range(16 * s, min(16 * s + 16, nb)))
                if not pages:
                    assert rep[b, s, g] == -1 and not sup[b, s, g].any()
                    continue
                l = int(rep[b, s, g])
                assert l in pages
                assert np.array_equal(sup[b, s, g], summ[bt[b, l], g]), "the representative is a copy of a member"
                # fp64 norms: no member is larger than the chosen one beyond fp32 rounding of a 128-term sum
                n2 = np.array([np.sum(f(summ[bt[b, p], g]).astype(np.float64) ** 2) for p in pages])
                assert n2[pages.index(l)] >= n2.max() * (1 - 1e-5)
                # ties in the fp32 norm go to the lowest page: every earlier member is strictly smaller
                n32 = [oracle.canon_dot(summ[bt[b, p], g], summ[bt[b, p], g]) for p in pages]
                assert all(n32[i] < n32[pages.index(l)] for i in range(pages.index(l)))
                assert all(n32[i] <= n32[pages.index(l)] for i in range(len(pages)))


def test_identical_pages_tie_to_the_lowest_page():
    w = make_workload(_spec(needles=0), seed=902)
    geo = geometry(w)
    q, K, V, bt, sl = host_arrays(w)
    K = K.copy()
    for b in range(geo.batch):               # every page of a sequence holds the same rows
        nb = (int(sl[b]) + 15) // 16
        for l in range(1, nb - 1):           # (the last page may be partial: its mean differs)
            K[bt[b, l]] = K[bt[b, 0]]
    summ = oracle.build_summaries(geo, K, bt, sl)
    sup, rep = oracle.build_super_summaries(geo, summ, bt, sl)
    n_full = ((sl + 15) // 16 - 1) // 16     # super-pages made of identical pages only
    for b in range(geo.batch):
        for s in range(int(n_full[b])):
            assert np.all(rep[b, s] == 16 * s)


def test_keeping_every_super_page_reproduces_the_exact_routing():
    w, geo, q, summ, sup, rep, bt, sl = _setup()
    P = 6
    exact = oracle.route(geo, q, summ, bt, sl, P)
    tl = oracle.route_two_level(geo, q, summ, sup, bt, sl, sup.shape[1], P)
    assert np.array_equal(tl.pages, exact.pages) and np.array_equal(tl.scores, exact.scores)


@pytest.mark.parametrize("P_super", [1, 2, 3])
def test_result_is_the_exact_top_P_inside_the_kept_super_pages(P_super):
    w, geo, q, summ, sup, rep, bt, sl = _setup()
    P = 6
    tl = oracle.route_two_level(geo, q, summ, sup, bt, sl, P_super, P)
    allr = oracle.route(geo, q, summ, bt, sl, 1, want_all_scores=True).all_scores
    G = geo.n_q_heads // geo.n_kv_heads
    for b in range(geo.batch):
        nb = (int(sl[b]) + 15) // 16
        ns = (nb + 15) // 16
        for h in range(geo.n_q_heads):
            # super-page selection: brute-force dominance under (score desc, index asc)
            ssc = np.array([oracle.canon_dot(q[b, h], sup[b, s, h // G]) for s in range(ns)])
            kept = [int(s) for s in tl.supers[b, h] if s >= 0]
            assert len(kept) == min(P_super, ns) and len(set(kept)) == len(kept)
            for s in kept:
                for t in range(ns):
                    if t not in kept:
                        assert (ssc[s] > ssc[t]) or (ssc[s] == ssc[t] and s < t)
            inside = [l for s in kept for l in range(16 * s, min(16 * s + 16, nb))]
            order = sorted(inside, key=lambda l: (-float(allr[b, h, l]), l))
            want = order[:P] + [-1] * max(0, P - len(order))
            assert tl.pages[b, h].tolist() == want
            got_sc = tl.scores[b, h][: min(P, len(order))]
            assert np.array_equal(got_sc, np.array([allr[b, h, l] for l in order[:P]], np.float32))


def test_needle_pages_are_recalled_with_a_fraction_of_the_super_pages():
    """Long sequence, 8 needles per KV head, P = 8: with as many super-pages kept as pages routed the exact
    routing's needle pages are found although only 8 of 64 super-pages are scanned."""
    w, geo, q, summ, sup, rep, bt, sl = _setup(seed=903, batch=1, seq_lens=(16384,), needles=8, P=8)
    P = 8
    exact = oracle.route(geo, q, summ, bt, sl, P)
    tl = oracle.route_two_level(geo, q, summ, sup, bt, sl, P, P)
    recall = []
    for h in range(geo.n_q_heads):
        e, t = set(exact.pages[0, h].tolist()), set(tl.pages[0, h].tolist())
        recall.append(len(e & t) / len(e))
    assert np.mean(recall) >= 0.9, recall
