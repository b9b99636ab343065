"""GPU parity at 32-token pages (the paper's sketch in Sec. 7 leaves the page size open): every step
through the C ABI against the oracle on the same seeded bytes, with the same bar as at 16 tokens -
summaries, radii, routed pages, scores, diagnostics, flags and lists bit for bit, floating-point
outputs within the tolerances of gpu_runner."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_runner import compare, run_gpu
from paper_2602_13804_b200 import binding as B
from test_gpu_certificate import compare_certified, run_certified
from test_gpu_solver import compare_entropic, compare_fw, run_entropic, run_fw
from test_gpu_two_level import _compare as compare_two_level, _run as run_two_level
from util import bits, geometry, host_arrays
from workloads import WorkloadSpec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def spec(**kw):
    base = dict(name="p32", config=9, batch=3, n_q_heads=8, n_kv_heads=2, P=3, K_c=40, page_size=32,
                seq_lens=(700, 333, 45), needles=3, needle_positions="uniform")
    base.update(kw)
    return WorkloadSpec(**base)


@pytest.mark.parametrize("hq,hkv", [(8, 2), (8, 1), (4, 4), (2, 1), (16, 1), (32, 2)])
@pytest.mark.parametrize("needles", [3, 0])
def test_small_ragged(hq, hkv, needles):
    w = make_workload(spec(n_q_heads=hq, n_kv_heads=hkv, needles=needles), seed=500 + hq * 10 + hkv)
    compare(w, run_gpu(w))


def test_lengths_around_page_and_block_boundaries():
    lens = (32 * 32 * 3 + 5, 32 * 32, 32 * 33 + 31, 1, 16, 17, 32, 33)
    w = make_workload(spec(batch=8, seq_lens=lens, P=8, K_c=100, needles=2), seed=521)
    compare(w, run_gpu(w))


def test_fewer_pages_than_P_and_fewer_tokens_than_Kc():
    w = make_workload(spec(batch=2, seq_lens=(70, 9), P=8, K_c=256), seed=522)
    g = run_gpu(w)
    compare(w, g)
    assert np.all(g.routed_pages[0, :, 3:] == -1) and np.all(g.routed_pages[1, :, 1:] == -1)
    assert g.diag_sparse["n_candidates"].reshape(2, 8)[0, 0] == 70


def test_dense_pass_for_every_unit_and_for_none():
    w = make_workload(spec(seq_lens=(2100, 999, 64), needles=0), seed=523)
    stats = compare(w, run_gpu(w, gap_threshold=math.inf), gap_threshold=math.inf)
    assert stats["fallback_fraction"] == 1.0
    compare(w, run_gpu(w, gap_threshold=-math.inf), gap_threshold=-math.inf)


def test_largest_candidate_count_and_both_block_sizes():
    # 64 pages of 32 tokens = 2048 scored tokens per unit (the limit), K_c = 700; 6 units take the 512-thread
    # shape, 600 the 128-thread one is excluded by the size (more than 64 tiles), 320 the 256-thread one
    w = make_workload(spec(batch=3, n_q_heads=2, n_kv_heads=1, seq_lens=(5000, 2500, 2049), P=64, K_c=700), seed=524)
    compare(w, run_gpu(w))
    w = make_workload(spec(batch=40, n_q_heads=8, n_kv_heads=2, seq_lens=tuple(200 + 37 * i for i in range(40)),
                           P=64, K_c=300, needles=2), seed=525)
    compare(w, run_gpu(w))


def test_many_units_take_the_128_thread_shape():
    w = make_workload(spec(batch=80, n_q_heads=8, n_kv_heads=2, seq_lens=tuple(90 + 21 * i for i in range(80)),
                           P=4, K_c=48, needles=2), seed=526)
    compare(w, run_gpu(w))


def test_engineered_ties():
    w = make_workload(spec(batch=2, seq_lens=(320, 192), needles=0, P=3, K_c=50), seed=527)
    k = w.k_cache.clone()
    bt = w.block_table
    for dst in (3, 4, 7):
        k[int(bt[0, dst])] = k[int(bt[0, 1])]
    k[int(bt[1, 2])] = k[int(bt[1, 0])]
    w.k_cache = k
    compare(w, run_gpu(w))


def test_non_native_strides():
    w = make_workload(spec(), seed=528)
    wd = w.to(DEV)
    k_alt = wd.k_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    v_alt = wd.v_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    wd.k_cache, wd.v_cache = k_alt, v_alt
    compare(w, run_gpu(wd))


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 4)])
def test_certified_step(hq, hkv):
    w = make_workload(spec(n_q_heads=hq, n_kv_heads=hkv, seq_lens=(1500, 700, 90), P=4, K_c=64), seed=530 + hq)
    compare_certified(w, run_certified(w))


@pytest.mark.parametrize("iters", [0, 3])
def test_iterative_solvers(iters):
    w = make_workload(spec(seq_lens=(900, 333, 45), P=4, K_c=48), seed=540)
    compare_entropic(w, run_entropic(w, iters), iters)
    compare_entropic(w, run_entropic(w, iters, fused=True), iters)
    compare_fw(w, run_fw(w, iters), iters)


@pytest.mark.parametrize("P_super", [1, 3])
def test_two_level_routing(P_super):
    w = make_workload(spec(batch=2, seq_lens=(32 * 16 * 5 + 40, 32 * 16 + 1), P=6, K_c=64), seed=550)
    compare_two_level(w, run_two_level(w, P_super, 6, 64), P_super, 6, 64)


def test_append_keeps_cache_and_summaries_in_step_with_a_rebuild():
    w = make_workload(spec(seq_lens=(64, 333, 31), needles=0), seed=560)   # the longest row leaves room to grow
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    summ = torch.zeros((shape.num_pool_pages, 2, 128), dtype=torch.bfloat16, device=DEV)
    radii = torch.zeros((shape.num_pool_pages, 2), dtype=torch.float32, device=DEV)
    B.vsa_build_page_summaries(shape, wd.k_cache, wd.block_table, wd.seq_lens, None, summ)
    B.vsa_build_page_radii(shape, wd.k_cache, summ, wd.block_table, wd.seq_lens, None, radii)
    q, K, V, bt, sl = host_arrays(w)
    K, V, bt, sl = K.copy(), V.copy(), bt.copy(), sl.copy()
    owned = set(bt[bt >= 0].tolist())
    free = [p for p in range(shape.num_pool_pages) if p not in owned]
    gen = torch.Generator().manual_seed(5)
    for step in range(3):
        kn = torch.randn((3, 2, 128), generator=gen).to(torch.bfloat16)
        vn = torch.randn((3, 2, 128), generator=gen).to(torch.bfloat16)
        for b in range(3):
            if sl[b] % 32 == 0:
                bt[b, sl[b] // 32] = free.pop()
            K[bt[b, sl[b] // 32], :, sl[b] % 32] = bits(kn[b])
            V[bt[b, sl[b] // 32], :, sl[b] % 32] = bits(vn[b])
        sl = sl + 1
        btd, sld = torch.from_numpy(bt).to(DEV), torch.from_numpy(sl).to(DEV)
        B.vsa_append_kv(shape, kn.to(DEV), vn.to(DEV), wd.k_cache, wd.v_cache, btd, sld, summ, radii)
    torch.cuda.synchronize()
    geo = geometry(w)
    assert np.array_equal(bits(wd.k_cache), K) and np.array_equal(bits(wd.v_cache), V)
    o_sum = oracle.build_summaries(geo, K, bt, sl)
    o_rad = oracle.build_radii(geo, K, o_sum, bt, sl)
    own = np.concatenate([bt[b, : -(-int(sl[b]) // 32)] for b in range(3)])
    assert np.array_equal(bits(summ)[own], o_sum[own])
    assert np.array_equal(radii.cpu().numpy()[own].view(np.uint32), o_rad[own].view(np.uint32))


def test_group_shared_entry_point_refuses_32_token_pages():
    w = make_workload(spec(), seed=570).to(DEV)
    shape = B.shape_of(w.q, w.k_cache, w.block_table)
    units = shape.batch * shape.n_q_heads
    summ = torch.zeros((shape.num_pool_pages, 2, 128), dtype=torch.bfloat16, device=DEV)
    out = torch.zeros((3, 8, 128), dtype=torch.float32, device=DEV)
    with pytest.raises(B.VsaError) as e:
        B.vsa_decode_step_group_shared(shape, w.q, summ, w.k_cache, w.v_cache, w.block_table, w.seq_lens, 3, 40,
                                       w.epsilon, w.gap_threshold, out, B.alloc_diag(units, DEV),
                                       torch.zeros((3, 2, 3), dtype=torch.int32, device=DEV),
                                       torch.zeros((units,), dtype=torch.int32, device=DEV),
                                       torch.zeros((1,), dtype=torch.int32, device=DEV),
                                       B.alloc_workspace(shape, 3, 40, B.VSA_WS_STEP, DEV))
    assert e.value.code == -2   # VSA_ERR_UNSUPPORTED_SHAPE
