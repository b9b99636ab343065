"""Pins of the CPU oracle against things other than itself: library routines, closed forms,
hand-derived values, brute force on tiny inputs, identities and bounds stated by the paper."""
import math

import numpy as np
import pytest
import torch

import oracle
from workloads import WorkloadSpec, make_workload
from util import bits, gathered_kv, geometry, host_arrays


def tiny_spec(**kw):
    base = dict(name="tiny", config=9, batch=2, n_q_heads=8, n_kv_heads=2, P=4, K_c=24,
                seq_lens=(300, 177), needles=3, needle_positions="uniform")
    base.update(kw)
    return WorkloadSpec(**base)


# ---------------------------------------------------------------- bf16 conversion

def test_bf16_rounding_matches_torch():
    g = torch.Generator().manual_seed(1)
    x = torch.randn(20000, generator=g) * 37.0
    # exact ties and neighbours of ties
    ties = torch.tensor([1.00390625, 1.01171875, -1.00390625, 3.0e38, 1e-40, 0.0, -0.0, 65280.0, 65408.0])
    x = torch.cat([x, ties])
    want = bits(x.to(torch.bfloat16))
    got = oracle.f32_to_bf16(x.numpy())
    assert np.array_equal(want, got)
    back = oracle.bf16_to_f32(got)
    assert np.array_equal(back, x.to(torch.bfloat16).float().numpy())


# ---------------------------------------------------------------- canonical fp32 dot

def _bf(v):
    return bits(torch.tensor(v, dtype=torch.float32).to(torch.bfloat16))


def test_canon_dot_small_integers_exact():
    rng = np.random.default_rng(0)
    x = rng.integers(-8, 9, 128).astype(np.float32)
    y = rng.integers(-8, 9, 128).astype(np.float32)
    # every partial sum is an integer below 2^24: any summation order is exact
    assert oracle.canon_dot(_bf(x), _bf(y)) == np.float32(int(x.astype(np.int64) @ y.astype(np.int64)))


def test_canon_dot_order_is_the_documented_tree():
    # products: chunk 0 -> 2^24, chunk 4 -> -2^24, chunk 8 -> 1, chunk 12 -> 1, rest 0.
    # halving tree: (p0+p8) = 2^24+1 -> rounds to 2^24 ; (p4+p12) = -2^24+1 exactly ;
    # then p0+p4 = 1.  A left-to-right sum over chunks would give 2, the exact value is 2.
    x = np.zeros(128, np.float32)
    y = np.zeros(128, np.float32)
    x[0], y[0] = 4096.0, 4096.0
    x[32], y[32] = 4096.0, -4096.0
    x[64], y[64] = 1.0, 1.0
    x[96], y[96] = 1.0, 1.0
    assert oracle.canon_dot(_bf(x), _bf(y)) == np.float32(1.0)
    # inside a chunk the even and the odd elements form two left-to-right chains:
    # even: ((2^24 + 1) + 1) - 2^24 = 0 (both +1 are rounded away), odd: 1; total 1.
    # One chain over all eight elements would give 0, the exact value is 3.
    x[:] = 0
    y[:] = 0
    x[0], y[0] = 4096.0, 4096.0
    x[1], y[1] = 1.0, 1.0
    x[2], y[2] = 1.0, 1.0
    x[4], y[4] = 1.0, 1.0
    x[6], y[6] = 4096.0, -4096.0
    assert oracle.canon_dot(_bf(x), _bf(y)) == np.float32(1.0)
    # the same four products spread so that the tree pairs them (c, c+8): (2^24 - 2^24) + (1 + 1)
    x[:] = 0
    y[:] = 0
    x[0], y[0] = 4096.0, 4096.0
    x[64], y[64] = 4096.0, -4096.0
    x[8], y[8] = 1.0, 1.0
    x[72], y[72] = 1.0, 1.0
    assert oracle.canon_dot(_bf(x), _bf(y)) == np.float32(2.0)


def test_canon_dot_close_to_fp64_and_symmetric():
    g = torch.Generator().manual_seed(2)
    for _ in range(200):
        x = torch.randn(128, generator=g).to(torch.bfloat16)
        y = torch.randn(128, generator=g).to(torch.bfloat16)
        exact = float(x.double() @ y.double())
        absdot = float(x.double().abs() @ y.double().abs())
        got = float(oracle.canon_dot(bits(x), bits(y)))
        # 7 + 4 additions deep: error <= 11 * 2^-24 * sum |x_i y_i|
        assert abs(got - exact) <= 11 * 2.0 ** -24 * absdot
        assert got == float(oracle.canon_dot(bits(y), bits(x)))


# ---------------------------------------------------------------- page summaries

def test_summaries_closed_forms():
    w = make_workload(tiny_spec(seq_lens=(64, 17), needles=0), seed=11)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    k = w.k_cache.clone()
    p_const, p_one = int(bt[0, 1]), int(bt[1, 1])   # a full page, and a page with 1 valid token
    row = torch.randn(2, 128).to(torch.bfloat16)
    k[p_const] = row[:, None, :]                    # 16 equal rows per head -> mean is that row
    K = bits(k)
    s = oracle.build_summaries(geo, K, bt, sl)
    assert np.array_equal(s[p_const], bits(row))
    # one valid token: the summary is that token (rows past the sequence end are ignored)
    assert np.array_equal(s[p_one], bits(k[p_one, :, 0, :]))
    # a page of the pool that no sequence owns is left untouched
    owned = set(bt[bt >= 0].tolist())
    free = next(i for i in range(geo.num_pool_pages) if i not in owned)
    assert not s[free].any()


def test_summaries_match_library_mean_within_one_ulp():
    w = make_workload(tiny_spec(needles=0), seed=12)
    q, K, V, bt, sl = host_arrays(w)
    s = oracle.bf16_to_f32(oracle.build_summaries(geometry(w), K, bt, sl))
    for b in range(2):
        T = int(sl[b])
        for l in range((T + 15) // 16):
            n = min(16, T - 16 * l)
            ref = w.k_cache[int(bt[b, l]), :, :n, :].double().mean(dim=1).numpy()
            got = s[int(bt[b, l])]
            assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30)


def test_summaries_first_page_updates_only_the_tail():
    w = make_workload(tiny_spec(needles=0), seed=13)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    full = oracle.build_summaries(geo, K, bt, sl)
    first = np.array([(300 - 1) // 16, (177 - 1) // 16], np.int32)
    part = oracle.build_summaries(geo, K, bt, sl, first_page=first)
    for b in range(2):
        last = int(bt[b, first[b]])
        assert np.array_equal(part[last], full[last])
        assert not part[int(bt[b, 0])].any()


# ---------------------------------------------------------------- selections

def _dominates(sa, ia, sb, ib):
    """(sa, ia) strictly precedes (sb, ib): score descending, index ascending."""
    return sa > sb or (sa == sb and ia < ib)


def test_route_is_the_top_P_of_the_total_order():
    w = make_workload(tiny_spec(), seed=21)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    r = oracle.route(geo, q, summ, bt, sl, P=4, want_all_scores=True)
    for b in range(2):
        nb = (int(sl[b]) + 15) // 16
        for h in range(8):
            sc = r.all_scores[b, h, :nb]
            chosen = r.pages[b, h].tolist()
            assert len(set(chosen)) == 4 and all(0 <= c < nb for c in chosen)
            rest = [l for l in range(nb) if l not in chosen]
            for c in chosen:
                for o in rest:
                    assert _dominates(sc[c], c, sc[o], o)
            # listed best first, and the same as a stable library sort on (-score, index)
            order = np.lexsort((np.arange(nb), -sc.astype(np.float64)))[:4]
            assert chosen == order.tolist()
            assert np.array_equal(r.scores[b, h], sc[order])
            # every score is the canonical dot of the query with the summary row
            g = h // 4
            l = chosen[0]
            assert sc[l] == oracle.canon_dot(q[b, h], summ[int(bt[b, l]), g])


def test_route_ties_take_the_lower_page_and_short_sequences_are_padded():
    w = make_workload(tiny_spec(seq_lens=(96, 40), needles=0), seed=22)
    k = w.k_cache.clone()
    bt = w.block_table
    # pages 1, 3 and 4 of sequence 0 are byte-identical: equal summaries, equal scores
    k[int(bt[0, 3])] = k[int(bt[0, 1])]
    k[int(bt[0, 4])] = k[int(bt[0, 1])]
    w.k_cache = k
    q, K, V, btn, sl = host_arrays(w)
    geo = geometry(w)
    summ = oracle.build_summaries(geo, K, btn, sl)
    r = oracle.route(geo, q, summ, btn, sl, P=4, want_all_scores=True)
    for h in range(8):
        chosen = r.pages[0, h].tolist()
        sc = r.all_scores[0, h]
        assert sc[1] == sc[3] == sc[4]
        tied = [c for c in chosen if c in (1, 3, 4)]
        assert tied == sorted(tied) and tied == [1, 3, 4][:len(tied)]
        # sequence 1 has 3 pages < P: all routed, then -1
        assert sorted(r.pages[1, h, :3].tolist()) == [0, 1, 2] and r.pages[1, h, 3] == -1
        assert r.scores[1, h, 3] == -np.inf


def test_negative_zero_scores_tie_with_positive_zero():
    w = make_workload(tiny_spec(batch=1, seq_lens=(64,), needles=0, n_q_heads=2, n_kv_heads=2), seed=23)
    k = torch.zeros_like(w.k_cache)
    bt = w.block_table
    k[int(bt[0, 2]), :, :, 0] = 1.0      # page 2: summary e_0 ; others: 0
    w.k_cache = k
    q = torch.zeros_like(w.q)
    q[0, 0, 0] = -1.0                    # head 0: page 2 scores -1, the rest +0 / -0 ties
    q[0, 1, 1] = -1.0                    # head 1: every product is -0 or +0: all tie
    w.q = q
    qn, K, V, btn, sl = host_arrays(w)
    geo = geometry(w)
    r = oracle.route(geo, qn, oracle.build_summaries(geo, K, btn, sl), btn, sl, P=3)
    assert r.pages[0, 0].tolist() == [0, 1, 3]
    assert r.pages[0, 1].tolist() == [0, 1, 2]


def test_token_selection_is_the_top_Kc_of_the_total_order():
    w = make_workload(tiny_spec(), seed=24)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    r = oracle.route(geo, q, oracle.build_summaries(geo, K, bt, sl), bt, sl, P=4)
    sp = oracle.sparse(geo, q, K, V, bt, sl, r.pages, K_c=24, epsilon=w.epsilon, gap_threshold=w.gap_threshold)
    for b in range(2):
        T = int(sl[b])
        for h in range(8):
            g = h // 4
            scored = {}
            for l in r.pages[b, h]:
                for t in range(16):
                    pos = int(l) * 16 + t
                    if l >= 0 and pos < T:
                        scored[pos] = oracle.canon_dot(q[b, h], K[int(bt[b, l]), g, t])
            S = [p for p in sp.cand_pos[b, h].tolist() if p >= 0]
            assert len(S) == min(24, len(scored)) == sp.n_candidates[b, h]
            rest = [p for p in scored if p not in S]
            for c in S:
                for o in rest:
                    assert _dominates(scored[c], c, scored[o], o)
            order = sorted(scored, key=lambda p: (-float(scored[p]), p))
            assert S == order[:len(S)]
            assert sp.s_max[b, h] == scored[order[0]]
            assert sp.delta12[b, h] == np.float32(scored[order[0]] - scored[order[1]])
            assert sp.delta[b, h] == np.float32(scored[order[0]] - scored[order[len(S)]])
            assert abs(sp.cand_weight[b, h].sum() - 1.0) < 1e-12


def test_token_ties_take_the_lower_position():
    w = make_workload(tiny_spec(batch=1, seq_lens=(64,), n_q_heads=2, n_kv_heads=1, needles=0), seed=25)
    k = w.k_cache.clone()
    bt = w.block_table
    # tokens 5, 18, 19 and 40 are the same vector, strongly aligned with head 0's query
    row = (3.0 * w.q[0, 0].float()).to(torch.bfloat16)
    for pos in (5, 18, 19, 40):
        k[int(bt[0, pos // 16]), 0, pos % 16] = row
    w.k_cache = k
    q, K, V, btn, sl = host_arrays(w)
    geo = geometry(w)
    pages = np.tile(np.arange(4, dtype=np.int32), (1, 2, 1))
    sp = oracle.sparse(geo, q, K, V, btn, sl, pages, K_c=3, epsilon=w.epsilon, gap_threshold=0.0)
    assert sp.cand_pos[0, 0].tolist() == [5, 18, 19]
    assert sp.delta[0, 0] == 0.0 and sp.delta12[0, 0] == 0.0      # best rejected token ties the best kept
    assert sp.fallback[0, 0] == 0                                  # strict "<" against threshold 0
    sp = oracle.sparse(geo, q, K, V, btn, sl, pages, K_c=3, epsilon=w.epsilon, gap_threshold=1e-3)
    assert sp.fallback[0, 0] == 1


# ---------------------------------------------------------------- dense attention = the definition

def test_dense_matches_library_sdpa_fp64():
    w = make_workload(tiny_spec(), seed=31)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    for eps in (w.epsilon, 1.0 / w.epsilon):
        eps32 = float(np.float32(eps))
        dn = oracle.dense(geo, q, K, V, bt, sl, eps32)
        for b in range(2):
            for h in range(8):
                k, v = gathered_kv(w, b, h // 4)
                qq = w.q[b, h].double()[None, None, None, :]
                ref = torch.nn.functional.scaled_dot_product_attention(
                    qq, k[None, None], v[None, None], scale=1.0 / eps32)[0, 0, 0]
                assert torch.allclose(torch.from_numpy(dn.out[b, h]), ref, rtol=0, atol=1e-12)
                ref_lse = torch.logsumexp(k @ w.q[b, h].double() / eps32, dim=0)
                assert abs(dn.lse[b, h] - float(ref_lse)) < 1e-10


def test_dense_brute_force_python_loops_tiny():
    w = make_workload(tiny_spec(batch=1, seq_lens=(19,), n_q_heads=2, n_kv_heads=1, needles=0), seed=32)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    dn = oracle.dense(geo, q, K, V, bt, sl, 2.5)
    for h in range(2):
        k, v = gathered_kv(w, 0, 0)
        qq = w.q[0, h].double().tolist()
        s = [sum(a * b for a, b in zip(qq, row)) / 2.5 for row in k.tolist()]
        z = sum(math.exp(x) for x in s)
        for e in range(128):
            y = sum(math.exp(x) * row[e] for x, row in zip(s, v.tolist())) / z
            assert abs(dn.out[0, h, e] - y) < 1e-12


def test_sparse_with_everything_routed_equals_dense():
    w = make_workload(tiny_spec(), seed=33)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    P = geo.max_pages_per_seq
    r = oracle.route(geo, q, oracle.build_summaries(geo, K, bt, sl), bt, sl, P=P)
    sp = oracle.sparse(geo, q, K, V, bt, sl, r.pages, K_c=P * 16, epsilon=w.epsilon, gap_threshold=1e30)
    dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon)
    assert np.allclose(sp.out, dn.out, rtol=0, atol=1e-13)
    assert np.allclose(sp.lse, dn.lse, rtol=0, atol=1e-12)
    assert np.array_equal(sp.n_candidates, np.repeat(sl[:, None], 8, axis=1))
    assert np.all(np.isposinf(sp.delta)) and not sp.fallback.any() and not sp.leak_bound.any()


# ---------------------------------------------------------------- leakage: identity and bounds

def test_two_term_split_and_leakage_bounds():
    """With S kept and the rest dropped:  y_dense - y_S = L * (y_off - y_S)  (the on-face /
    off-face split of the main theorem's proof, whose on-face term vanishes for the plain
    softmax), L <= (T - |S|) exp(-Delta_S / eps) and per token a_j <= exp(-Delta_S / eps)
    (Cor. 1 with c = 1), and |y_dense - y_S| <= L * diam(V) (off-face readout lemma)."""
    for seed, needles in ((41, 3), (42, 0)):
        w = make_workload(tiny_spec(needles=needles), seed=seed)
        q, K, V, bt, sl = host_arrays(w)
        geo = geometry(w)
        r = oracle.route(geo, q, oracle.build_summaries(geo, K, bt, sl), bt, sl, P=4)
        sp = oracle.sparse(geo, q, K, V, bt, sl, r.pages, K_c=24, epsilon=w.epsilon, gap_threshold=w.gap_threshold)
        dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon, cand_pos=sp.cand_pos)
        for b in range(2):
            T = int(sl[b])
            for h in range(8):
                L = dn.true_leak[b, h]
                lhs = dn.out[b, h] - sp.out[b, h]
                rhs = L * (dn.y_off[b, h] - sp.out[b, h])
                assert np.max(np.abs(lhs - rhs)) < 1e-12
                nS = int(sp.n_candidates[b, h])
                bound = (T - nS) * math.exp(-dn.true_gap[b, h] / w.epsilon)
                assert 0.0 <= L <= bound * (1 + 1e-12)
                k, v = gathered_kv(w, b, h // 4)
                diam = float(torch.cdist(v, v).max())
                assert np.linalg.norm(lhs) <= L * diam * (1 + 1e-12) + 1e-13
                # per-token bound, recomputed from library softmax weights
                a = torch.softmax(k @ w.q[b, h].double() / w.epsilon, dim=0).numpy()
                mask = np.ones(T, bool)
                mask[[p for p in sp.cand_pos[b, h] if p >= 0]] = False
                assert abs(a[mask].sum() - L) < 1e-12
                assert np.all(a[mask] <= math.exp(-dn.true_gap[b, h] / w.epsilon) * (1 + 1e-12))
                # the in-pass bound is min(1, (T-|S|) exp(-delta/eps)) with the fp32 proxy
                want = min(1.0, (T - nS) * math.exp(-float(sp.delta[b, h]) / w.epsilon))
                assert abs(sp.leak_bound[b, h] - want) <= 1e-12 * max(1.0, want)


def test_planted_needles_pass_the_gap_test_and_iid_keys_do_not():
    planted = make_workload(tiny_spec(seq_lens=(2048, 1500), needles=4, P=8, K_c=64), seed=51)
    iid = make_workload(tiny_spec(seq_lens=(2048, 1500), needles=0, P=8, K_c=64), seed=52)
    for w, want in ((planted, 0), (iid, 1)):
        q, K, V, bt, sl = host_arrays(w)
        st = oracle.decode_step(geometry(w), q, K, V, bt, sl, 8, 64, w.epsilon, w.gap_threshold)
        assert np.all(st.sparse.fallback == want)
        if want:   # flagged units carry the dense output
            dn = oracle.dense(geometry(w), q, K, V, bt, sl, w.epsilon)
            assert np.array_equal(st.out, dn.out)
        else:      # certified units are close to dense: leakage is exponentially small
            dn = oracle.dense(geometry(w), q, K, V, bt, sl, w.epsilon)
            assert np.max(np.abs(st.out - dn.out)) < 1e-3


# ---------------------------------------------------------------- gap statistic s(1) - s(2)

def test_gap_statistic_follows_the_extreme_value_law():
    """App. B: for iid N(0,1) scores sqrt(2 log M) (s(1) - s(2)) => Exp(1).  Scores <q,k> with
    iid N(0, I) keys are iid N(0, |q|^2), so the statistic is scaled by |q|."""
    T = 4096
    w = make_workload(tiny_spec(batch=4, n_q_heads=32, n_kv_heads=8, seq_lens=(T,) * 4, needles=0), seed=61)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    pages = np.tile(np.arange(T // 16, dtype=np.int32), (4, 32, 1))
    sp = oracle.sparse(geo, q, K, V, bt, sl, pages, K_c=2, epsilon=w.epsilon, gap_threshold=0.0)
    qn = np.linalg.norm(oracle.bf16_to_f32(q).astype(np.float64), axis=-1)
    stat = math.sqrt(2 * math.log(T)) * sp.delta12 / qn
    # Exp(1): mean 1, P(X > 1) = e^-1; 128 samples, finite-M bias is a few percent
    assert 0.75 < stat.mean() < 1.25
    assert 0.22 < (stat > 1.0).mean() < 0.52
    assert stat.min() >= 0.0
