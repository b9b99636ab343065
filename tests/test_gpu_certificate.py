"""GPU parity of the routing certificate (vsa_build_page_radii / vsa_decode_step_certified) against the
oracle on the same seeded bytes.  Radii, the bound over the un-routed pages, the certified gap and the
certified flag - which decides the fallback - are single-rounded fp32 arithmetic in a fixed order and
must match bit for bit; leak_bound_cert is an fp32 exponential compared with a relative tolerance."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2602_13804_b200 import binding as B
from gpu_runner import check_out
from util import geometry, host_arrays
from workloads import WorkloadSpec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def spec(**kw):
    base = dict(name="t", config=9, batch=3, n_q_heads=8, n_kv_heads=2, P=4, K_c=40,
                seq_lens=(700, 333, 90), needles=3, needle_positions="uniform")
    base.update(kw)
    return WorkloadSpec(**base)


def run_certified(w):
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    units = shape.batch * shape.n_q_heads
    P, K_c = w.spec.P, w.spec.K_c
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    radii = torch.full((shape.num_pool_pages, shape.n_kv_heads), -1.0, dtype=torch.float32, device=DEV)
    B.vsa_build_page_radii(shape, wd.k_cache, summ, wd.block_table, wd.seq_lens, None, radii)
    out = torch.full((shape.batch, shape.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag, cert = B.alloc_diag(units, DEV), B.alloc_cert(units, DEV)
    flist = torch.full((units,), -1, dtype=torch.int32, device=DEV)
    fcount = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    routed = torch.full((shape.batch, shape.n_q_heads, P), -7, dtype=torch.int32, device=DEV)
    ws = B.alloc_workspace(shape, P, K_c, B.VSA_WS_STEP_CERTIFIED, DEV)
    B.vsa_decode_step_certified(shape, wd.q, summ, radii, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, P, K_c,
                                w.epsilon, w.gap_threshold, out, diag, cert, routed, flist, fcount, ws)
    torch.cuda.synchronize()
    n = int(fcount.item())
    return dict(out=out.cpu().numpy(), diag={k: v.numpy() for k, v in B.diag_to_dict(diag).items()},
                cert={k: v.numpy() for k, v in B.cert_to_dict(cert).items()}, radii=radii.cpu().numpy(),
                routed=routed.cpu().numpy(), fallback=np.sort(flist[:n].cpu().numpy()))


def compare_certified(w, g):
    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    Bn, H = geo.batch, geo.n_q_heads
    summ = oracle.build_summaries(geo, K, bt, sl)
    rad = oracle.build_radii(geo, K, summ, bt, sl)
    owned = np.concatenate([bt[b, : -(-int(sl[b]) // geo.page_size)] for b in range(Bn)])
    assert np.array_equal(g["radii"][owned].view(np.uint32), rad[owned].view(np.uint32)), "radii differ"
    untouched = np.ones(geo.num_pool_pages, bool)
    untouched[owned] = False
    assert np.all(g["radii"][untouched] == -1.0)
    rt = oracle.route(geo, q, summ, bt, sl, w.spec.P, want_all_scores=True)
    assert np.array_equal(g["routed"], rt.pages)
    sp = oracle.sparse(geo, q, K, V, bt, sl, rt.pages, w.spec.K_c, w.epsilon, w.gap_threshold)
    ce = oracle.certify(geo, q, rad, bt, sl, rt, sp, w.epsilon, w.gap_threshold)
    c = g["cert"]
    assert np.array_equal(c["ub_unrouted"].reshape(Bn, H).view(np.uint32), ce.ub_unrouted.view(np.uint32)), "bounds differ"
    assert np.array_equal(c["delta_cert"].reshape(Bn, H).view(np.uint32), ce.delta_cert.view(np.uint32)), "gaps differ"
    assert np.array_equal(c["certified"].reshape(Bn, H), ce.certified)
    lb = c["leak_bound_cert"].reshape(Bn, H).astype(np.float64)
    assert np.all(np.abs(lb - ce.leak_cert) <= 1e-3 * ce.leak_cert + 1e-37)
    # the certified gap decides the fallback; the other diagnostics are those of the plain step
    want_fb = ((ce.certified == 0) & (sp.n_candidates < sl[:, None])).astype(np.int32)
    d = g["diag"]
    assert np.array_equal(d["fallback"].reshape(Bn, H), want_fb)
    assert np.array_equal(g["fallback"], np.nonzero(want_fb.reshape(-1))[0])
    for name, want in (("delta", sp.delta), ("delta12", sp.delta12), ("s_max", sp.s_max)):
        assert np.array_equal(d[name].reshape(Bn, H), want), name
    assert np.array_equal(d["n_candidates"].reshape(Bn, H), sp.n_candidates)
    # outputs: sparse rows where certified, dense rows where the unit fell back
    flat = want_fb.reshape(-1).astype(bool)
    out = g["out"].reshape(Bn * H, -1)
    if (~flat).any():
        check_out(out[~flat], sp.out.reshape(Bn * H, -1)[~flat], "certified rows")
    if flat.any():
        dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon, unit_mask=want_fb)
        check_out(out[flat], dn.out.reshape(Bn * H, -1)[flat], "fallback rows")
    return ce, sp, want_fb


@pytest.mark.parametrize("hq,hkv", [(8, 2), (8, 1), (4, 4), (4, 2)])
def test_certified_step_matches_the_oracle(hq, hkv):
    w = make_workload(spec(n_q_heads=hq, n_kv_heads=hkv), seed=400 + hq + hkv)
    ce, sp, fb = compare_certified(w, run_certified(w))
    assert np.all(ce.delta_cert <= sp.delta)


def test_certificate_passes_for_planted_heads_and_fails_for_flat_ones():
    # strong needles: the best score clears every ball bound; needle-free heads cannot be certified
    w = make_workload(spec(seq_lens=(2000, 1500, 900), P=8, K_c=64, needles=4), seed=410)
    ce, sp, fb = compare_certified(w, run_certified(w))
    assert ce.certified.any()
    w0 = make_workload(spec(seq_lens=(2000, 1500, 900), P=8, K_c=64, needles=0), seed=411)
    ce0, sp0, fb0 = compare_certified(w0, run_certified(w0))
    assert not ce0.certified.any() and fb0.all()


def test_everything_routed_and_ragged_tails():
    # P covers every page of the short sequences: no un-routed page, the certified gap is the proxy gap
    w = make_workload(spec(seq_lens=(60, 17, 1), P=4, K_c=20), seed=412)
    g = run_certified(w)
    ce, sp, fb = compare_certified(w, g)
    assert np.all(np.isneginf(ce.ub_unrouted)) and np.array_equal(ce.delta_cert, sp.delta)


def test_incremental_radius_update_of_the_last_page():
    w = make_workload(spec(needles=0), seed=413).to(DEV)
    shape = B.shape_of(w.q, w.k_cache, w.block_table)
    summ = torch.zeros((shape.num_pool_pages, 2, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, w.k_cache, w.block_table, w.seq_lens, None, summ)
    full = torch.zeros((shape.num_pool_pages, 2), dtype=torch.float32, device=DEV)
    B.vsa_build_page_radii(shape, w.k_cache, summ, w.block_table, w.seq_lens, None, full)
    part = torch.zeros_like(full)
    first = torch.tensor([(700 - 1) // 16, (333 - 1) // 16, (90 - 1) // 16], dtype=torch.int32, device=DEV)
    B.vsa_build_page_radii(shape, w.k_cache, summ, w.block_table, w.seq_lens, first, part)
    torch.cuda.synchronize()
    for b in range(3):
        last = int(w.block_table[b, int(first[b])])
        assert torch.equal(part[last], full[last]) and not part[int(w.block_table[b, 0])].any()


def test_wide_block_table_and_many_units():
    # 2500 pages per sequence with 160 units: the 256-thread kernel with 16 page scores per thread
    w = make_workload(spec(batch=20, n_q_heads=8, n_kv_heads=2, seq_lens=(40000,) + (900,) * 19, P=16, K_c=128,
                           needles=6), seed=414)
    compare_certified(w, run_certified(w))


def test_more_units_than_resident_blocks_take_the_128_thread_shape():
    # 320 units, ragged; then 2500 pages per sequence (32 page scores and radii per thread at 128 threads)
    lens = tuple(150 + 41 * i for i in range(40))
    w = make_workload(spec(batch=40, n_q_heads=8, n_kv_heads=2, seq_lens=lens, P=8, K_c=64, needles=3), seed=415)
    compare_certified(w, run_certified(w))
    w = make_workload(spec(batch=40, n_q_heads=8, n_kv_heads=4, seq_lens=(40000,) + (700,) * 39, P=16, K_c=128,
                           needles=6), seed=416)
    compare_certified(w, run_certified(w))


def test_append_keeps_cache_summaries_and_radii_in_step_with_a_full_rebuild():
    """Three appended tokens per sequence (the first one opens a new page for sequence 0): rows,
    summaries and radii must equal what the oracle builds from scratch on the grown cache."""
    w = make_workload(spec(seq_lens=(160, 333, 15), needles=0), seed=415)
    # room for the growth: the generator sizes block-table rows for the initial lengths
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    radii = torch.zeros((shape.num_pool_pages, shape.n_kv_heads), dtype=torch.float32, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    B.vsa_build_page_radii(shape, wd.k_cache, summ, wd.block_table, wd.seq_lens, None, radii)
    q, K, V, bt, sl = host_arrays(w)
    K, V, sl = K.copy(), V.copy(), sl.copy()
    geo = geometry(w)
    gen = torch.Generator().manual_seed(9)
    lens = wd.seq_lens.clone()
    bt = bt.copy()
    free = sorted(set(range(geo.num_pool_pages)) - set(int(x) for x in bt.reshape(-1) if x >= 0))
    for step in range(3):
        for b in range(3):          # the scheduler's part: a fresh page when the new token opens one
            if int(sl[b]) % 16 == 0:
                bt[b, int(sl[b]) // 16] = free.pop()
        wd.block_table = torch.from_numpy(bt).to(DEV)
        k_new = torch.randn((3, 2, 128), generator=gen).to(torch.bfloat16)
        v_new = torch.randn((3, 2, 128), generator=gen).to(torch.bfloat16)
        lens = lens + 1
        B.vsa_append_kv(shape, k_new.to(DEV), v_new.to(DEV), wd.k_cache, wd.v_cache, wd.block_table, lens, summ, radii)
        kb = k_new.view(torch.int16).numpy().view(np.uint16)
        vb = v_new.view(torch.int16).numpy().view(np.uint16)
        for b in range(3):
            pos = int(sl[b])
            K[bt[b, pos // 16], :, pos % 16] = kb[b]
            V[bt[b, pos // 16], :, pos % 16] = vb[b]
        sl = sl + 1
    torch.cuda.synchronize()
    from util import bits
    assert np.array_equal(bits(wd.k_cache), K) and np.array_equal(bits(wd.v_cache), V)
    o_sum = oracle.build_summaries(geo, K, bt, sl)
    o_rad = oracle.build_radii(geo, K, o_sum, bt, sl)
    owned = np.concatenate([bt[b, : (int(sl[b]) + 15) // 16] for b in range(3)])
    assert np.array_equal(bits(summ)[owned], o_sum[owned])
    assert np.array_equal(radii.cpu().numpy()[owned].view(np.uint32), o_rad[owned].view(np.uint32))


def test_expansion_retries_the_refused_units_with_more_pages_before_the_dense_pass():
    """Two to twenty needles per (sequence, kv head) against six routed pages: units with few needles
    certify in the first pass, the others miss needle pages and are refused; with P_expand = 24 every
    needle page is routed and all but one of them pass; that one goes to the dense pass.  The composite
    expectation is assembled from the oracle's parts."""
    P, P2, K_c = 6, 24, 64
    w = make_workload(spec(batch=6, seq_lens=(3000, 2000, 700, 1500, 2600, 900), P=P, K_c=K_c, needles=(2, 20)),
                      seed=421)
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    units = shape.batch * shape.n_q_heads
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    radii = torch.zeros((shape.num_pool_pages, shape.n_kv_heads), dtype=torch.float32, device=DEV)
    B.vsa_build_page_radii(shape, wd.k_cache, summ, wd.block_table, wd.seq_lens, None, radii)
    out = torch.full((shape.batch, shape.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag, cert = B.alloc_diag(units, DEV), B.alloc_cert(units, DEV)
    flist = torch.full((units,), -1, dtype=torch.int32, device=DEV)
    fcount = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    routed = torch.full((shape.batch, shape.n_q_heads, P2), -7, dtype=torch.int32, device=DEV)
    ws = B.alloc_workspace(shape, P2, K_c, B.VSA_WS_STEP_EXPAND, DEV)
    for _ in range(2):      # twice: the retry list and its counter are reset by the call itself
        B.vsa_decode_step_certified_expand(shape, wd.q, summ, radii, wd.k_cache, wd.v_cache, wd.block_table,
                                           wd.seq_lens, P, P2, K_c, w.epsilon, w.gap_threshold, out, diag, cert,
                                           routed, flist, fcount, ws)
    torch.cuda.synchronize()

    q, K, V, bt, sl = host_arrays(w)
    geo = geometry(w)
    Bn, H = geo.batch, geo.n_q_heads
    o_sum = oracle.build_summaries(geo, K, bt, sl)
    o_rad = oracle.build_radii(geo, K, o_sum, bt, sl)

    def one_pass(p):
        rt = oracle.route(geo, q, o_sum, bt, sl, p, want_all_scores=True)
        sp = oracle.sparse(geo, q, K, V, bt, sl, rt.pages, K_c, w.epsilon, w.gap_threshold)
        ce = oracle.certify(geo, q, o_rad, bt, sl, rt, sp, w.epsilon, w.gap_threshold)
        refused = (ce.certified == 0) & (sp.n_candidates < sl[:, None])
        return rt, sp, ce, refused

    # the loop: P, 2P, ... up to P2; a unit's state is that of the last pass it took part in
    passes, p = [], P
    while True:
        passes.append((p,) + one_pass(p))
        if p >= P2:
            break
        p = min(2 * p, P2)
    assert len(passes) == 3, "6 -> 12 -> 24 pages"
    active = np.ones((Bn, H), bool)            # units that run the current pass
    last_pass = np.zeros((Bn, H), int)
    for k, (_, _, _, _, refused) in enumerate(passes):
        last_pass[active] = k
        active = active & refused
    final_fb = active
    ref1 = passes[0][4]
    assert ref1.any() and not ref1.all(), "the workload should refuse some units with P pages and keep others"
    assert (ref1 & ~final_fb).any(), "the expansion should rescue some units"
    assert final_fb.any(), "and leave at least one to the dense pass"
    assert (last_pass == 1).any() and (last_pass == 2).any(), "both retry passes should end some unit"

    def pick(field):
        out_ = None
        for k, (_, rt, sp, ce, _) in enumerate(passes):
            a = field(rt, sp, ce)
            out_ = a.copy() if out_ is None else np.where(last_pass == k, a, out_)
        return out_

    want_routed = np.full((Bn, H, P2), -1, np.int32)
    for k, (pk, rt, _, _, _) in enumerate(passes):
        rows = last_pass == k
        want_routed[rows, :pk] = rt.pages[rows]
    assert np.array_equal(routed.cpu().numpy(), want_routed)
    c = {k: v.numpy().reshape(Bn, H) for k, v in B.cert_to_dict(cert).items()}
    d = {k: v.numpy().reshape(Bn, H) for k, v in B.diag_to_dict(diag).items()}
    for name in ("delta_cert", "ub_unrouted"):
        want = pick(lambda rt, sp, ce: getattr(ce, name))
        assert np.array_equal(c[name].view(np.uint32), want.view(np.uint32)), name
    assert np.array_equal(c["certified"], pick(lambda rt, sp, ce: ce.certified))
    assert np.array_equal(d["n_candidates"], pick(lambda rt, sp, ce: sp.n_candidates))
    assert np.array_equal(d["delta"], pick(lambda rt, sp, ce: sp.delta))
    assert np.array_equal(d["fallback"], final_fb.astype(np.int32))
    def pick_out():
        o = None
        for k, (_, _, sp, _, _) in enumerate(passes):
            o = sp.out.copy() if o is None else np.where((last_pass == k)[..., None], sp.out, o)
        return o
    sp_last_out = pick_out().reshape(Bn * H, -1)
    n = int(fcount.item())
    assert np.array_equal(np.sort(flist[:n].cpu().numpy()), np.nonzero(final_fb.reshape(-1))[0])
    got = out.cpu().numpy().reshape(Bn * H, -1)
    sparse_rows, dense_rows = (~final_fb).reshape(-1), final_fb.reshape(-1)
    check_out(got[sparse_rows], sp_last_out[sparse_rows], "units certified by their last sparse pass")
    if dense_rows.any():
        dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon, unit_mask=final_fb.astype(np.int32))
        check_out(got[dense_rows], dn.out.reshape(Bn * H, -1)[dense_rows], "units that fell back")


def test_certified_step_with_bad_inputs_sets_status_without_trapping():
    w = make_workload(spec(seq_lens=(300, 177, 90), needles=0), seed=430)
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    units = shape.batch * shape.n_q_heads
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    radii = torch.zeros((shape.num_pool_pages, shape.n_kv_heads), dtype=torch.float32, device=DEV)
    B.vsa_build_page_radii(shape, wd.k_cache, summ, wd.block_table, wd.seq_lens, None, radii)
    sl = wd.seq_lens.clone()
    sl[1] = shape.max_pages_per_seq * 16 + 5          # longer than its block-table row
    sl[2] = 0                                         # empty
    out = torch.full((shape.batch, shape.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag, cert = B.alloc_diag(units, DEV), B.alloc_cert(units, DEV)
    cert.fill_(-1)
    flist = torch.full((units,), -1, dtype=torch.int32, device=DEV)
    fcount = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    routed = torch.full((shape.batch, shape.n_q_heads, 4), -7, dtype=torch.int32, device=DEV)
    ws = B.alloc_workspace(shape, 4, 40, B.VSA_WS_STEP_CERTIFIED, DEV)
    B.vsa_decode_step_certified(shape, wd.q, summ, radii, wd.k_cache, wd.v_cache, wd.block_table, sl, 4, 40,
                                w.epsilon, -math.inf, out, diag, cert, routed, flist, fcount, ws)
    # the append skips the same sequences
    k_new = torch.ones((3, 2, 128), dtype=torch.bfloat16, device=DEV)
    before = wd.k_cache.clone()
    B.vsa_append_kv(shape, k_new, k_new, wd.k_cache, wd.v_cache, wd.block_table, sl, summ, radii)
    torch.cuda.synchronize()
    d = B.diag_to_dict(diag)
    st = d["status"].view(3, 8)
    assert st[0].eq(0).all() and st[1].eq(2).all() and st[2].eq(2).all()
    o = out.cpu().numpy()
    assert np.isfinite(o[0]).all() and not o[1:].any()
    c = B.cert_to_dict(cert)
    assert c["certified"].view(3, 8)[1:].eq(0).all() and c["delta_cert"].view(3, 8)[1:].eq(0).all()
    assert int(fcount.item()) == 0
    assert np.all(routed.cpu().numpy()[1:] == -1)
    changed = (wd.k_cache != before).flatten(1).any(1).nonzero().flatten().tolist()
    assert changed == [int(wd.block_table[0, (300 - 1) // 16])]      # only sequence 0's last page was written
