"""Pins of the oracle at 32-token pages (the paper's system sketch, Sec. 7, leaves the page size open;
16 is the size every other pin uses).  What fixes the 32-token results independently of the oracle's
own page loop: closed forms and a library mean for the summaries, a brute-force top-P over scores
recomputed one by one, and the re-paging identity - the token-level steps (token routing, candidate
softmax, diagnostics, dense attention) do not know where page boundaries fall, so cutting every
32-token page into two 16-token pages and routing both halves must reproduce every output bit for bit."""
import numpy as np
import torch

import oracle
from util import bits, geometry, host_arrays
from workloads import WorkloadSpec, make_workload


def _w(seed=3, **kw):
    base = dict(name="p32", config=9, batch=3, n_q_heads=8, n_kv_heads=2, P=3, K_c=40, page_size=32,
                seq_lens=(700, 333, 45), needles=3, needle_positions="uniform")
    base.update(kw)
    return make_workload(WorkloadSpec(**base), seed=seed)


def _halved(w):
    """The same cache cut into 16-token pages: pool page p becomes pages 2p and 2p + 1."""
    geo32 = geometry(w)
    k, v = w.k_cache.cpu(), w.v_cache.cpu()
    pool, hkv, bs, d = k.shape
    assert bs == 32

    def cut(t):
        return t.reshape(pool, hkv, 2, 16, d).permute(0, 2, 1, 3, 4).reshape(pool * 2, hkv, 16, d).contiguous()

    bt = w.block_table.cpu().numpy().astype(np.int32)
    bt16 = np.full((bt.shape[0], bt.shape[1] * 2), -1, np.int32)
    bt16[:, 0::2] = np.where(bt >= 0, 2 * bt, -1)
    bt16[:, 1::2] = np.where(bt >= 0, 2 * bt + 1, -1)
    geo16 = oracle.Geometry(batch=geo32.batch, n_q_heads=geo32.n_q_heads, n_kv_heads=geo32.n_kv_heads,
                            max_pages_per_seq=bt16.shape[1], num_pool_pages=pool * 2, head_dim=d, page_size=16)
    return geo16, bits(cut(k)), bits(cut(v)), bt16


def test_summaries_closed_forms_at_32_tokens():
    w = _w(seq_lens=(96, 33, 64), needles=0)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    k = w.k_cache.clone()
    p_const, p_one, p_int = int(bt[0, 1]), int(bt[1, 1]), int(bt[2, 0])
    row = torch.randn(2, 128).to(torch.bfloat16)
    k[p_const] = row[:, None, :]                      # 32 equal rows per head -> the mean is that row
    ints = torch.randint(-3, 4, (2, 32, 128)).float()
    k[p_int] = ints.to(torch.bfloat16)                # small integers: sum and sum / 32 are exact in fp32 and bf16
    s = oracle.build_summaries(geo, bits(k), bt, sl)
    assert np.array_equal(s[p_const], bits(row))
    assert np.array_equal(s[p_one], bits(k[p_one, :, 0, :]))   # one valid token
    want = (ints.sum(dim=1) / 32.0)
    assert torch.equal(want.to(torch.bfloat16).float(), want)   # representable, so the pin is exact
    assert np.array_equal(oracle.bf16_to_f32(s[p_int]), want.numpy())


def test_summaries_match_library_mean_within_one_ulp_at_32_tokens():
    w = _w(needles=0, seed=4)
    q, K, V, bt, sl = host_arrays(w)
    s = oracle.bf16_to_f32(oracle.build_summaries(geometry(w), K, bt, sl))
    for b in range(3):
        T = int(sl[b])
        for l in range((T + 31) // 32):
            n = min(32, T - 32 * l)
            ref = w.k_cache[int(bt[b, l]), :, :n, :].double().mean(dim=1).numpy()
            assert np.all(np.abs(s[int(bt[b, l])] - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30)


def test_route_is_a_brute_force_top_P_at_32_tokens():
    w = _w(seed=5)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    P = 5
    r = oracle.route(geo, q, summ, bt, sl, P)
    for b in range(geo.batch):
        nb = (int(sl[b]) + 31) // 32
        for h in range(geo.n_q_heads):
            sc = np.array([oracle.canon_dot(q[b, h], summ[int(bt[b, l]), h // 4]) for l in range(nb)], np.float32)
            order = np.lexsort((np.arange(nb), -sc.astype(np.float64)))[:P]
            want = np.full(P, -1, np.int32)
            want[:len(order)] = order
            assert np.array_equal(r.pages[b, h], want)


def _expand(pages32, sl):
    """routed 32-token pages -> the 16-token pages that cover the same tokens (entries past the end dropped)"""
    B, H, P = pages32.shape
    out = np.full((B, H, 2 * P), -1, np.int32)
    for b in range(B):
        nb16 = (int(sl[b]) + 15) // 16
        for h in range(H):
            for j, l in enumerate(pages32[b, h]):
                if l < 0:
                    continue
                out[b, h, 2 * j] = 2 * l
                if 2 * l + 1 < nb16:
                    out[b, h, 2 * j + 1] = 2 * l + 1
    return out


def test_token_level_steps_do_not_depend_on_the_page_size():
    w = _w(seed=6)
    q, K, V, bt, sl = host_arrays(w)
    geo32 = geometry(w)
    geo16, K16, V16, bt16 = _halved(w)
    r = oracle.route(geo32, q, oracle.build_summaries(geo32, K, bt, sl), bt, sl, w.spec.P)
    for thr in (w.gap_threshold, 1e30, 0.0):
        a = oracle.sparse(geo32, q, K, V, bt, sl, r.pages, w.spec.K_c, w.epsilon, thr)
        c = oracle.sparse(geo16, q, K16, V16, bt16, sl, _expand(r.pages, sl), w.spec.K_c, w.epsilon, thr)
        for f in ("out", "delta", "delta12", "s_max", "lse", "leak_bound", "n_candidates", "fallback", "cand_pos",
                  "cand_weight", "best_rejected"):
            assert np.array_equal(getattr(a, f), getattr(c, f)), f
    d32 = oracle.dense(geo32, q, K, V, bt, sl, w.epsilon)
    d16 = oracle.dense(geo16, q, K16, V16, bt16, sl, w.epsilon)
    assert np.array_equal(d32.out, d16.out) and np.array_equal(d32.lse, d16.lse)
    # the candidates really come from the routed 32-token pages
    for b in range(geo32.batch):
        for h in range(geo32.n_q_heads):
            pos = a.cand_pos[b, h]
            pos = pos[pos >= 0]
            assert set((pos // 32).tolist()) <= set(r.pages[b, h].tolist())
            assert len(pos) == min(w.spec.K_c, sum(min(32, int(sl[b]) - 32 * l) for l in r.pages[b, h] if l >= 0))


def test_radius_covers_every_row_at_32_tokens():
    w = _w(seed=7)
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    summ = oracle.build_summaries(geo, K, bt, sl)
    rad = oracle.build_radii(geo, K, summ, bt, sl)
    Kf, mu = oracle.bf16_to_f32(K).astype(np.float64), oracle.bf16_to_f32(summ).astype(np.float64)
    for b in range(geo.batch):
        T = int(sl[b])
        for l in range((T + 31) // 32):
            p, n = int(bt[b, l]), min(32, T - 32 * l)
            for g in range(geo.n_kv_heads):
                dist = np.linalg.norm(Kf[p, g, :n] - mu[p, g], axis=1).max()
                slack = 2.0 ** -12 * np.linalg.norm(mu[p, g])
                assert dist <= rad[p, g] <= 1.0011 * dist + 1.001 * slack


def test_planted_needles_are_found_at_32_tokens():
    w = _w(seed=8, seq_lens=(2000, 1500, 900), P=6, K_c=64)
    q, K, V, bt, sl = host_arrays(w)
    st = oracle.decode_step(geometry(w), q, K, V, bt, sl, w.spec.P, w.spec.K_c, w.epsilon, w.gap_threshold)
    dn = oracle.dense(geometry(w), q, K, V, bt, sl, w.epsilon)
    assert not st.sparse.fallback.any()
    assert np.abs(st.out - dn.out).max() < 1e-3
