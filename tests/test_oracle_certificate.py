"""Pins of the oracle's routing certificate (orc_build_radii / orc_certify): the ball bound is a
construction of this library (the paper only asks for "certificates" that the screened set is
right, App. E), so what pins it is the property it claims - no token outside the candidate set
scores above s(1) - delta_cert - checked by brute force in fp64 over every token, plus closed
forms for degenerate pages."""
import numpy as np
import torch

import oracle
from util import geometry, host_arrays
from workloads import WorkloadSpec, make_workload


def _workload(seed=5, **kw):
    base = dict(name="t", config=9, batch=3, n_q_heads=4, n_kv_heads=2, P=3, K_c=20,
                seq_lens=(333, 150, 49), needles=2, needle_positions="uniform")
    base.update(kw)
    return make_workload(WorkloadSpec(**base), seed=seed)


def _f64(bits_):
    return oracle.bf16_to_f32(bits_).astype(np.float64)


def _all(w):
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    rad = oracle.build_radii(geo, K, summ, bt, sl)
    rt = oracle.route(geo, q, summ, bt, sl, w.spec.P, want_all_scores=True)
    sp = oracle.sparse(geo, q, K, V, bt, sl, rt.pages, w.spec.K_c, w.epsilon, w.gap_threshold)
    ce = oracle.certify(geo, q, rad, bt, sl, rt, sp, w.epsilon, w.gap_threshold)
    return geo, q, K, V, bt, sl, summ, rad, rt, sp, ce


def test_radius_covers_every_row_and_is_tight():
    w = _workload()
    geo, q, K, V, bt, sl, summ, rad, *_ = _all(w)
    Kf, mu = _f64(K), _f64(summ)
    for b in range(geo.batch):
        T = int(sl[b])
        for l in range((T + 15) // 16):
            p, n = int(bt[b, l]), min(16, T - 16 * l)
            for g in range(geo.n_kv_heads):
                dist = np.linalg.norm(Kf[p, g, :n] - mu[p, g], axis=1).max()
                slack = 2.0 ** -12 * np.linalg.norm(mu[p, g])
                assert dist <= rad[p, g]
                assert rad[p, g] <= 1.0011 * dist + 1.001 * slack


def test_single_row_page_has_the_closed_form_radius():
    # a page with one valid row: the stored mean is that row, r = 0, rhat = 2^-12 |k|
    w = _workload(seq_lens=(17, 1, 33))
    geo, q, K, V, bt, sl, summ, rad, *_ = _all(w)
    Kf = _f64(K)
    for b, l in ((0, 1), (1, 0), (2, 2)):
        p = int(bt[b, l])
        for g in range(geo.n_kv_heads):
            want = 2.0 ** -12 * np.linalg.norm(Kf[p, g, 0])
            assert abs(rad[p, g] - want) <= 2e-7 * want


def test_no_token_outside_the_candidates_beats_the_certified_level():
    """Brute force over every token of every sequence, exact fp64 scores."""
    for seed, needles in ((5, 2), (6, 0), (7, 5)):
        w = _workload(seed=seed, needles=needles)
        geo, q, K, V, bt, sl, summ, rad, rt, sp, ce = _all(w)
        Kf, qf = _f64(K), _f64(q)
        G = geo.n_q_heads // geo.n_kv_heads
        for b in range(geo.batch):
            T = int(sl[b])
            rows = np.concatenate([Kf[int(bt[b, l])] for l in range((T + 15) // 16)], axis=1)[:, :T]   # [Hkv, T, d]
            for h in range(geo.n_q_heads):
                s_all = rows[h // G] @ qf[b, h]
                inside = np.zeros(T, bool)
                inside[sp.cand_pos[b, h][sp.cand_pos[b, h] >= 0]] = True
                level = float(sp.s_max[b, h]) - float(ce.delta_cert[b, h])
                routed = np.zeros(T, bool)
                for l in rt.pages[b, h][rt.pages[b, h] >= 0]:
                    routed[16 * l: 16 * l + 16] = True
                if (~routed).any():
                    # never scored: the exact score is below the ball bound, with no tolerance
                    assert s_all[~routed].max() <= float(ce.ub_unrouted[b, h])
                    assert float(ce.ub_unrouted[b, h]) <= level + 1e-4      # level = s1 - (s1 - max(...)) in fp32
                if (routed & ~inside).any():
                    # scored and rejected: the level is their fp32 score, the exact one differs by rounding
                    assert s_all[routed & ~inside].max() <= level + 2e-4
                if (~inside).any():
                    # the certified gap never exceeds the proxy gap (which ignores un-routed pages)
                    assert ce.delta_cert[b, h] <= sp.delta[b, h]
                else:
                    assert np.isposinf(ce.delta_cert[b, h])
                assert int(ce.certified[b, h]) == int(ce.delta_cert[b, h] >= np.float32(w.gap_threshold))


def test_certified_leakage_bound_holds_for_the_dense_softmax():
    w = _workload(seed=8, needles=3)
    geo, q, K, V, bt, sl, summ, rad, rt, sp, ce = _all(w)
    dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon, cand_pos=sp.cand_pos)
    assert np.all(dn.true_leak <= ce.leak_cert + 1e-12)
    assert np.all(ce.leak_cert <= 1.0)
    # with needles the certificate is not vacuous for the planted heads
    assert (ce.leak_cert < 1e-3).any()


def test_all_pages_routed_reduces_to_the_proxy_gap():
    w = _workload(seq_lens=(40, 30, 16), P=4)
    geo, q, K, V, bt, sl, summ, rad, rt, sp, ce = _all(w)
    assert np.all(np.isneginf(ce.ub_unrouted))
    assert np.array_equal(ce.delta_cert, sp.delta)


def test_hand_built_page_of_identical_rows():
    """Two pages; page 1 holds sixteen copies of a bf16-exact row a and is not routed (P = 1).  Its
    bound is <q, a> + qn * 2^-12 |a| with qn = |q| (1 + 2^-20), in fp32."""
    w = _workload(batch=1, n_q_heads=1, n_kv_heads=1, seq_lens=(32,), P=1, K_c=4, needles=0)
    a = torch.linspace(-1, 1, 128).to(torch.bfloat16)
    k = w.k_cache.clone()
    k[int(w.block_table[0, 1]), 0] = a
    k[int(w.block_table[0, 0]), 0] = (4.0 * w.q[0, 0].float()).to(torch.bfloat16)    # page 0 wins the routing
    w.k_cache = k
    geo, q, K, V, bt, sl, summ, rad, rt, sp, ce = _all(w)
    assert rt.pages[0, 0, 0] == 0
    af, qf = a.double().numpy(), _f64(q)[0, 0]
    want = af @ qf + np.linalg.norm(qf) * (1 + 2.0 ** -20) * 2.0 ** -12 * np.linalg.norm(af)
    assert abs(float(ce.ub_unrouted[0, 0]) - want) <= 1e-5 * max(1.0, abs(want))
    assert float(ce.delta_cert[0, 0]) == float(np.float32(sp.s_max[0, 0]) - max(np.float32(sp.best_rejected[0, 0]),
                                                                               ce.ub_unrouted[0, 0]))
