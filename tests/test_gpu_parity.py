"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded bytes.  Discrete results (summaries, routed pages, candidate-derived diagnostics,
fallback flags and lists) must match bit for bit; floating-point outputs within 1e-2 max-abs
and 5e-3 relative L2."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2602_13804_b200 import binding as B
from gpu_runner import check_out, compare, run_gpu
from util import bits, geometry, host_arrays
from workloads import WorkloadSpec, config_spec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def spec(**kw):
    base = dict(name="t", config=9, batch=2, n_q_heads=8, n_kv_heads=2, P=4, K_c=24,
                seq_lens=(300, 177), needles=3, needle_positions="uniform")
    base.update(kw)
    return WorkloadSpec(**base)


# ---------------------------------------------------------------- small shapes, every group size

@pytest.mark.parametrize("hq,hkv", [(8, 2), (8, 1), (4, 2), (4, 4), (16, 2)])
@pytest.mark.parametrize("needles", [3, 0])
def test_small_ragged(hq, hkv, needles):
    w = make_workload(spec(n_q_heads=hq, n_kv_heads=hkv, needles=needles), seed=100 + hq * 10 + hkv)
    stats = compare(w, run_gpu(w))
    assert 0.0 <= stats["fallback_fraction"] <= 1.0


@pytest.mark.parametrize("mode", ["per_qhead_round_robin", "unit_literal"])
def test_other_needle_layouts(mode):
    # needles aligned to one head of a group at a time (the heads of a group then route to different
    # pages: no page sharing), and the literal unit-vector needle that iid keys out-score
    w = make_workload(spec(seq_lens=(2500, 900), needles=8, P=6, K_c=64, needle_mode=mode), seed=220)
    compare(w, run_gpu(w))


@pytest.mark.parametrize("hq,hkv", [(16, 1), (32, 1), (32, 2)])
def test_multi_query_groups_of_16_and_32(hq, hkv):
    """Multi-query shapes (16 or 32 query heads per KV head): scan and dense pass split the group into
    sub-groups of 8 that read the same KV head; everything must still match the oracle, the dense pass
    included (threshold +inf sends every unit there)."""
    w = make_workload(spec(seq_lens=(900, 333), n_q_heads=hq, n_kv_heads=hkv, needles=3), seed=230 + hq + hkv)
    compare(w, run_gpu(w))
    compare(w, run_gpu(w, gap_threshold=math.inf), gap_threshold=math.inf)


def test_several_tiles_and_ragged_tail():
    # 5 sequences with lengths around page and 32-page-block boundaries, several scan blocks
    lens = (16 * 32 * 3 + 5, 16 * 32, 16 * 33 + 15, 1, 16)
    w = make_workload(spec(batch=5, seq_lens=lens, n_q_heads=8, n_kv_heads=2, P=8, K_c=40, needles=2), seed=201)
    compare(w, run_gpu(w))


def test_routing_fewer_pages_than_P_and_fewer_tokens_than_Kc():
    w = make_workload(spec(seq_lens=(40, 7), P=8, K_c=128), seed=202)
    g = run_gpu(w)
    compare(w, g)
    assert np.all(g.routed_pages[0, :, 3:] == -1) and np.all(g.routed_pages[1, :, 1:] == -1)
    assert np.all(np.isposinf(g.diag_sparse["delta"])) and not g.diag_sparse["fallback"].any()
    assert g.diag_sparse["n_candidates"].reshape(2, 8)[0, 0] == 40


def test_engineered_ties_pages_and_tokens():
    w = make_workload(spec(seq_lens=(160, 96), needles=0, P=3, K_c=20), seed=203)
    k = w.k_cache.clone()
    bt = w.block_table
    for dst in (3, 4, 7):                      # pages 1, 3, 4, 7 of sequence 0 byte-identical
        k[int(bt[0, dst])] = k[int(bt[0, 1])]
    k[int(bt[1, 2])] = k[int(bt[1, 0])]        # pages 0 and 2 of sequence 1 identical
    w.k_cache = k
    g = run_gpu(w)
    compare(w, g)
    # all-equal scores: every page ties, lowest indices win
    w2 = make_workload(spec(seq_lens=(200, 64), needles=0, P=5, K_c=17), seed=204)
    w2.k_cache = torch.zeros_like(w2.k_cache)
    g2 = run_gpu(w2)
    compare(w2, g2)
    assert g2.routed_pages[0, 0].tolist() == [0, 1, 2, 3, 4]


def test_thresholds_minus_inf_never_and_plus_inf_always():
    w = make_workload(spec(needles=0), seed=205)
    g = run_gpu(w, gap_threshold=-math.inf)
    compare(w, g, gap_threshold=-math.inf)
    assert len(g.fallback_units) == 0
    g = run_gpu(w, gap_threshold=math.inf)
    stats = compare(w, g, gap_threshold=math.inf)
    assert stats["fallback_fraction"] == 1.0


def test_literal_small_epsilon():
    w = make_workload(spec(seq_lens=(700, 333), needles=4, P=6, K_c=48), seed=206)
    eps = float(np.float32(1.0 / math.sqrt(128.0)))
    compare(w, run_gpu(w, epsilon=eps), epsilon=eps)


def test_non_native_strides():
    # cache stored as [pool, page, kv_head, d]: token stride = Hkv * d, head stride = d
    w = make_workload(spec(), seed=207)
    wd = w.to(DEV)
    k_alt = wd.k_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    v_alt = wd.v_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert k_alt.stride(2) == 2 * 128 and k_alt.stride(1) == 128
    wd.k_cache, wd.v_cache = k_alt, v_alt
    compare(w, run_gpu(wd))


def test_dense_baseline_all_units_matches_definition():
    w = make_workload(spec(seq_lens=(1000, 513), n_q_heads=8, n_kv_heads=2), seed=208).to(DEV)
    shape = B.shape_of(w.q, w.k_cache, w.block_table)
    out = torch.full((2, 8, 128), float("nan"), dtype=torch.float32, device=DEV)
    ws = B.alloc_workspace(shape, 0, 0, B.VSA_WS_DENSE, DEV)
    B.vsa_dense_decode_fallback(shape, w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, None, None, w.epsilon,
                                out, None, ws)
    q, K, V, bt, sl = host_arrays(w)
    dn = oracle.dense(geometry(w), q, K, V, bt, sl, w.epsilon)
    check_out(out.cpu().numpy(), dn.out, "dense baseline")


def test_bad_block_table_entry_and_bad_length_set_status_without_trapping():
    w = make_workload(spec(seq_lens=(300, 177), needles=0), seed=209).to(DEV)
    shape = B.shape_of(w.q, w.k_cache, w.block_table)
    units = 16
    summ = torch.zeros((shape.num_pool_pages, 2, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, w.k_cache, w.block_table, w.seq_lens, None, summ)
    routed = torch.zeros((2, 8, 4), dtype=torch.int32, device=DEV)
    routed[:, :, :] = torch.tensor([0, 1, 2, 3], dtype=torch.int32, device=DEV)
    bt = w.block_table.clone()
    bt[0, 2] = shape.num_pool_pages + 5            # sequence 0 routes through a bad entry
    sl = w.seq_lens.clone()
    sl[1] = shape.max_pages_per_seq * 16 + 1       # sequence 1 claims more tokens than its row holds
    out = torch.full((2, 8, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag = B.alloc_diag(units, DEV)
    fl = torch.zeros(units, dtype=torch.int32, device=DEV)
    fc = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.vsa_sparse_decode(shape, w.q, w.k_cache, w.v_cache, bt, sl, routed, 4, 24, w.epsilon, w.gap_threshold, out,
                        diag, fl, fc)
    torch.cuda.synchronize()
    d = B.diag_to_dict(diag)
    assert d["status"].view(2, 8)[0].tolist() == [1] * 8 and d["status"].view(2, 8)[1].tolist() == [2] * 8
    assert not out.cpu().numpy().any() and int(fc.item()) == 0
    # routing with the same bad inputs: bad pages score -inf, the over-long sequence routes nothing
    rp = torch.zeros((2, 8, 4), dtype=torch.int32, device=DEV)
    ws = B.alloc_workspace(shape, 4, 24, B.VSA_WS_ROUTE, DEV)
    B.vsa_route_pages(shape, w.q, summ, bt, sl, 4, rp, None, ws)
    torch.cuda.synchronize()
    assert 2 not in rp[0].cpu().numpy() and np.all(rp[1].cpu().numpy() == -1)


def test_dense_pass_fails_the_units_of_a_sequence_with_an_entry_outside_the_pool():
    """Every page of a listed sequence is needed by the dense pass: one block-table entry outside the pool
    (bounds-checked, never dereferenced) must give status BAD_PAGE and a zero row for all heads of that
    sequence, and leave the other sequence's result equal to the definition."""
    w = make_workload(spec(seq_lens=(1000, 513), n_q_heads=8, n_kv_heads=2), seed=208).to(DEV)
    shape = B.shape_of(w.q, w.k_cache, w.block_table)
    bt = w.block_table.clone()
    bt[0, 40] = -3
    out = torch.full((2, 8, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag = B.alloc_diag(16, DEV)
    ws = B.alloc_workspace(shape, 0, 0, B.VSA_WS_DENSE, DEV)
    B.vsa_dense_decode_fallback(shape, w.q, w.k_cache, w.v_cache, bt, w.seq_lens, None, None, w.epsilon,
                                out, diag, ws)
    torch.cuda.synchronize()
    d = B.diag_to_dict(diag)
    assert d["status"].view(2, 8)[0].tolist() == [1] * 8
    assert not out[0].cpu().numpy().any()
    q, K, V, bt_h, sl = host_arrays(w)
    dn = oracle.dense(geometry(w), q, K, V, bt_h, sl, w.epsilon)
    check_out(out[1].cpu().numpy(), dn.out[1], "dense baseline, intact sequence")


def test_incremental_summary_update_of_the_last_page():
    w = make_workload(spec(needles=0), seed=210).to(DEV)
    shape = B.shape_of(w.q, w.k_cache, w.block_table)
    full = torch.zeros((shape.num_pool_pages, 2, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, w.k_cache, w.block_table, w.seq_lens, None, full)
    part = torch.zeros_like(full)
    first = torch.tensor([(300 - 1) // 16, (177 - 1) // 16], dtype=torch.int32, device=DEV)
    B.vsa_build_page_summaries(shape, w.k_cache, w.block_table, w.seq_lens, first, part)
    torch.cuda.synchronize()
    for b in range(2):
        last = int(w.block_table[b, int(first[b])])
        assert torch.equal(part[last], full[last])
        assert not part[int(w.block_table[b, 0])].any()


def test_host_buffer_step_matches_device_step():
    from paper_2602_13804_b200 import SparsePagedDecoder
    w = make_workload(spec(seq_lens=(900, 640), needles=2, P=6, K_c=48), seed=211)
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    dec = SparsePagedDecoder(shape, 6, 48, w.epsilon, w.gap_threshold, device=DEV, host_io=True)
    summ = dec.build_summaries(wd.k_cache, wd.block_table, wd.seq_lens)
    out_dev = dec.step(wd.q, summ, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens).clone()
    q_host = w.q.pin_memory()
    out_host = dec.step_host(q_host, summ, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens)
    torch.cuda.synchronize()
    assert torch.equal(out_host, out_dev.cpu())
    assert torch.equal(dec.diag_host, dec.diag.cpu())
    # pageable host buffers take the staged-copy route; page-locked ones above are used in place
    diag_ref = dec.diag.cpu().clone()
    out_pg = torch.full(out_host.shape, float("nan"), dtype=torch.float32)
    diag_pg = torch.zeros_like(dec.diag_host, pin_memory=False)
    assert not out_pg.is_pinned() and not w.q.is_pinned()
    B.vsa_decode_step_host(shape, w.q, dec.q_dev, summ, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens, 6, 48,
                           w.epsilon, w.gap_threshold, out_pg, dec.out, diag_pg, dec.diag, dec.routed_pages,
                           dec.fallback_list, dec.fallback_count, dec.ws)
    torch.cuda.synchronize()
    assert torch.equal(out_pg, out_dev.cpu()) and torch.equal(diag_pg, diag_ref)
    q, K, V, bt, sl = host_arrays(w)
    st = oracle.decode_step(geometry(w), q, K, V, bt, sl, 6, 48, w.epsilon, w.gap_threshold)
    check_out(out_host.numpy(), st.out, "host step")


def test_largest_routing_sizes():
    # P = 128, K_c = 2048: eight token scores per thread, four page-list entries per lane
    w = make_workload(spec(batch=3, n_q_heads=8, n_kv_heads=2, seq_lens=(40000, 5000, 2100), P=128, K_c=2048,
                           needles=40), seed=212)
    compare(w, run_gpu(w), dense_sample=8)
    # more units than SMs with the same sizes: the 256-thread shape
    w = make_workload(spec(batch=20, n_q_heads=8, n_kv_heads=1, seq_lens=(3000,) * 20, P=128, K_c=1500,
                           needles=10), seed=213)
    compare(w, run_gpu(w), dense_sample=8)


def test_more_units_than_resident_blocks():
    # 640 and 320 units: beyond two 256-thread blocks per SM the kernel takes its 128-thread shape, here
    # with eight token scores per thread (P = 64) and with two (P = 8); ragged lengths, several waves
    lens = tuple(200 + 37 * i for i in range(80))
    w = make_workload(spec(batch=80, n_q_heads=8, n_kv_heads=2, seq_lens=lens, P=64, K_c=300, needles=4), seed=216)
    compare(w, run_gpu(w), dense_sample=8)
    w = make_workload(spec(batch=40, n_q_heads=8, n_kv_heads=1, seq_lens=lens[:40], P=8, K_c=40, needles=2), seed=217)
    compare(w, run_gpu(w), dense_sample=8)
    # one long sequence among many short ones, table wider than 32 page scores per thread: the pool cannot
    # hold 80 sequences of that length, so the 128-thread shape with the selection in shared memory runs
    w = make_workload(spec(batch=80, n_q_heads=4, n_kv_heads=2, seq_lens=(70000,) + (600,) * 79, P=16, K_c=100,
                           needles=5), seed=218)
    assert w.block_table.shape[0] * w.block_table.shape[1] > w.k_cache.shape[0]
    compare(w, run_gpu(w), dense_sample=4)


def test_block_table_wider_than_the_register_select():
    # 9000 pages per sequence: beyond 32 scores per thread at 256 threads, within it at 512;
    # batch 40 x 4 heads = 160 units > SMs forces the 256-thread kernel and its shared-memory select
    w = make_workload(spec(batch=40, n_q_heads=4, n_kv_heads=4, seq_lens=(144000,) + (600,) * 39, P=16, K_c=100,
                           needles=5), seed=214)
    compare(w, run_gpu(w), dense_sample=4)
    # few units: 512 threads, 18 scores per thread rounded up to the 32-wide register select
    w = make_workload(spec(batch=1, n_q_heads=4, n_kv_heads=2, seq_lens=(144000,), P=16, K_c=100, needles=5),
                      seed=215)
    compare(w, run_gpu(w), dense_sample=2)


# ---------------------------------------------------------------- the named configurations

def test_config0_full():
    w = make_workload(config_spec(0), device=DEV)
    stats = compare(w, run_gpu(w))
    assert stats["fallback_fraction"] == 0.0       # planted needles: the support gap is positive
    eps = float(np.float32(1.0 / math.sqrt(128.0)))  # the literal small temperature, parity only
    compare(w, run_gpu(w, epsilon=eps), epsilon=eps)


def test_config0_round_robin_needles():
    w = make_workload(config_spec(0, needle_mode="per_qhead_round_robin"), device=DEV)
    compare(w, run_gpu(w))


def test_config1_full_one_layer():
    w = make_workload(config_spec(1), device=DEV)
    stats = compare(w, run_gpu(w))
    assert stats["fallback_fraction"] == 0.0


@pytest.mark.parametrize("batch,T", [(1, 131072), (16, 8192), (1, 4096)])
def test_config2_sweep_points(batch, T):
    w = make_workload(config_spec(2, batch=batch, T=T), device=DEV, sub=int(math.log2(T)))
    compare(w, run_gpu(w), dense_sample=16)


def test_config3_fallback_regime_reduced():
    w = make_workload(config_spec(3, batch=4, T=8192, needle_seqs=1), device=DEV)
    stats = compare(w, run_gpu(w))
    assert stats["fallback_fraction"] == 0.75


def test_config3_full_sampled_dense():
    w = make_workload(config_spec(3), device=DEV)
    stats = compare(w, run_gpu(w), dense_sample=24)
    assert stats["fallback_fraction"] == 0.75      # 12 of 16 sequences have no planted structure


def test_config4_ragged_gqa8_reduced():
    w = make_workload(config_spec(4, batch=6, ragged_T=(300, 5000)), device=DEV)
    compare(w, run_gpu(w), dense_sample=16)


def test_config4_full_sampled_dense():
    w = make_workload(config_spec(4), device=DEV)
    compare(w, run_gpu(w), dense_sample=16)
