"""GPU parity at head dimensions 64 and 256 (the paper's method is shape-agnostic, Sec. 7): summaries,
routing, the fused sparse pass and the dense pass through the C ABI against the oracle on the same seeded
bytes, with the same bar as at 128 - discrete results bit for bit, floating-point outputs within the
tolerances of gpu_runner.  The iterative solves, the certificate, two-level and group-shared routing and
the token append exist at 128 only and must refuse other dimensions."""
import math
import random

import numpy as np
import pytest
import torch

from gpu_runner import compare, run_gpu
from paper_2602_13804_b200 import binding as B
from workloads import WorkloadSpec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
DIMS = (64, 256)


def spec(d, **kw):
    base = dict(name=f"d{d}", config=9, batch=3, n_q_heads=8, n_kv_heads=2, P=4, K_c=40, head_dim=d,
                epsilon=math.sqrt(d), seq_lens=(700, 333, 45), needles=3, needle_positions="uniform")
    base.update(kw)
    return WorkloadSpec(**base)


@pytest.mark.parametrize("d", DIMS)
@pytest.mark.parametrize("hq,hkv", [(8, 2), (8, 1), (4, 4), (2, 1), (16, 1), (32, 2)])
@pytest.mark.parametrize("needles", [3, 0])
def test_small_ragged(d, hq, hkv, needles):
    w = make_workload(spec(d, n_q_heads=hq, n_kv_heads=hkv, needles=needles), seed=700 + d + hq * 10 + hkv)
    compare(w, run_gpu(w))


@pytest.mark.parametrize("d", DIMS)
def test_lengths_around_page_and_block_boundaries(d):
    lens = (16 * 32 * 3 + 5, 16 * 32, 16 * 33 + 15, 1, 15, 16, 17)
    w = make_workload(spec(d, batch=7, seq_lens=lens, P=8, K_c=100, needles=2), seed=720 + d)
    compare(w, run_gpu(w))


@pytest.mark.parametrize("d", DIMS)
def test_dense_pass_for_every_unit_and_for_none(d):
    w = make_workload(spec(d, seq_lens=(2100, 999, 64), needles=0), seed=730 + d)
    stats = compare(w, run_gpu(w, gap_threshold=math.inf), gap_threshold=math.inf)
    assert stats["fallback_fraction"] == 1.0
    compare(w, run_gpu(w, gap_threshold=-math.inf), gap_threshold=-math.inf)


@pytest.mark.parametrize("d", DIMS)
def test_pages_of_32_tokens(d):
    w = make_workload(spec(d, page_size=32, seq_lens=(1500, 700, 33), P=3, K_c=64), seed=740 + d)
    compare(w, run_gpu(w))
    compare(w, run_gpu(w, gap_threshold=math.inf), gap_threshold=math.inf)


@pytest.mark.parametrize("d", DIMS)
def test_largest_candidate_count_every_block_size_and_a_wide_table(d):
    # 6 units: 512 threads; 320 units: 256 threads; 640 units with few pages: 128 threads; 70k tokens: the
    # selection staged in shared memory
    w = make_workload(spec(d, batch=3, n_q_heads=2, n_kv_heads=1, seq_lens=(5000, 2500, 2049), P=128, K_c=700), seed=750 + d)
    compare(w, run_gpu(w))
    w = make_workload(spec(d, batch=40, seq_lens=tuple(200 + 37 * i for i in range(40)), P=64, K_c=300, needles=2),
                      seed=751 + d)
    compare(w, run_gpu(w))
    w = make_workload(spec(d, batch=80, seq_lens=tuple(90 + 21 * i for i in range(80)), P=4, K_c=48, needles=2),
                      seed=752 + d)
    compare(w, run_gpu(w))
    w = make_workload(spec(d, batch=2, seq_lens=(70000, 900), P=16, K_c=128), seed=753 + d)
    compare(w, run_gpu(w), dense_sample=4)


@pytest.mark.parametrize("d", DIMS)
def test_engineered_ties_and_non_native_strides(d):
    w = make_workload(spec(d, batch=2, seq_lens=(160, 96), needles=0, P=3, K_c=20), seed=760 + d)
    k = w.k_cache.clone()
    bt = w.block_table
    for dst in (3, 4, 7):
        k[int(bt[0, dst])] = k[int(bt[0, 1])]
    k[int(bt[1, 2])] = k[int(bt[1, 0])]
    w.k_cache = k
    compare(w, run_gpu(w))
    w2 = make_workload(spec(d), seed=761 + d)
    wd = w2.to(DEV)
    wd.k_cache = wd.k_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    wd.v_cache = wd.v_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    compare(w2, run_gpu(wd))


@pytest.mark.parametrize("d", DIMS)
def test_random_shapes(d):
    rng = random.Random(900 + d)
    for case in range(10):
        G = rng.choice([1, 2, 4, 8, 16])
        hkv = rng.choice([1, 2, 4])
        hq = G * hkv
        batch = rng.randint(1, max(1, 400 // hq))
        page = rng.choice([16, 32])
        P = rng.choice([p for p in (1, 2, 5, 8, 16, 31, 32, 64) if p * page <= 2048])
        K_c = min(rng.choice([1, 7, 40, 100, 256, 700]), P * page)
        lens = tuple(rng.choice([1, page - 1, page, page + 1, rng.randint(1, 600), rng.randint(1, 3000)]) for _ in range(batch))
        w = make_workload(spec(d, batch=batch, n_q_heads=hq, n_kv_heads=hkv, P=P, K_c=K_c, page_size=page, seq_lens=lens,
                               needles=rng.choice([0, 1, 3])), seed=26000 + d + case)
        compare(w, run_gpu(w), dense_sample=4)


@pytest.mark.parametrize("d", DIMS)
def test_entry_points_that_exist_at_128_only_refuse(d):
    w = make_workload(spec(d), seed=770 + d).to(DEV)
    shape = B.shape_of(w.q, w.k_cache, w.block_table)
    units = shape.batch * shape.n_q_heads
    summ = torch.zeros((shape.num_pool_pages, 2, d), dtype=torch.bfloat16, device=DEV)
    radii = torch.zeros((shape.num_pool_pages, 2), dtype=torch.float32, device=DEV)
    out = torch.zeros((3, 8, d), dtype=torch.float32, device=DEV)
    diag = B.alloc_diag(units, DEV)
    routed = torch.zeros((3, 8, 4), dtype=torch.int32, device=DEV)
    flist = torch.zeros((units,), dtype=torch.int32, device=DEV)
    fcount = torch.zeros((1,), dtype=torch.int32, device=DEV)
    ws = torch.zeros((1 << 22,), dtype=torch.uint8, device=DEV)
    calls = [
        lambda: B.vsa_build_page_radii(shape, w.k_cache, summ, w.block_table, w.seq_lens, None, radii),
        lambda: B.vsa_decode_step_certified(shape, w.q, summ, radii, w.k_cache, w.v_cache, w.block_table, w.seq_lens, 4,
                                            40, w.epsilon, w.gap_threshold, out, diag, B.alloc_cert(units, DEV), routed,
                                            flist, fcount, ws),
        lambda: B.vsa_decode_step_entropic(shape, w.q, summ, w.k_cache, w.v_cache, w.block_table, w.seq_lens, 4, 40,
                                           w.epsilon, w.gap_threshold, 2, out, diag, B.alloc_solve(units, DEV), routed,
                                           flist, fcount, ws),
        lambda: B.vsa_decode_step_group_shared(shape, w.q, summ, w.k_cache, w.v_cache, w.block_table, w.seq_lens, 4, 40,
                                               w.epsilon, w.gap_threshold, out, diag,
                                               torch.zeros((3, 2, 4), dtype=torch.int32, device=DEV), flist, fcount, ws),
    ]
    for call in calls:
        with pytest.raises(B.VsaError) as e:
            call()
        assert e.value.code == -2   # VSA_ERR_UNSUPPORTED_SHAPE


@pytest.mark.parametrize("d", DIMS)
def test_host_buffer_step_and_workspace_free_routing(d):
    import oracle
    from gpu_runner import check_out
    from paper_2602_13804_b200 import SparsePagedDecoder
    from util import geometry, host_arrays
    w = make_workload(spec(d, batch=2, seq_lens=(900, 640), needles=2, P=6, K_c=48), seed=780 + d)
    wd = w.to(DEV)
    shape = B.shape_of(wd.q, wd.k_cache, wd.block_table)
    dec = SparsePagedDecoder(shape, 6, 48, w.epsilon, w.gap_threshold, device=DEV, host_io=True)
    summ = dec.build_summaries(wd.k_cache, wd.block_table, wd.seq_lens)
    out_dev = dec.step(wd.q, summ, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens).clone()
    out_host = dec.step_host(w.q.pin_memory(), summ, wd.k_cache, wd.v_cache, wd.block_table, wd.seq_lens)
    torch.cuda.synchronize()
    assert out_host.shape[-1] == d and torch.equal(out_host, out_dev.cpu())
    q, K, V, bt, sl = host_arrays(w)
    st = oracle.decode_step(geometry(w), q, K, V, bt, sl, 6, 48, w.epsilon, w.gap_threshold)
    check_out(out_host.numpy(), st.out, "host step")
    routed = torch.full((2, 8, 6), -7, dtype=torch.int32, device=DEV)
    scores = torch.zeros((2, 8, 6), dtype=torch.float32, device=DEV)
    B.vsa_route_pages_static(shape, wd.q, summ, wd.block_table, wd.seq_lens, 6, routed, scores)
    torch.cuda.synchronize()
    assert np.array_equal(routed.cpu().numpy(), st.route.pages) and np.array_equal(scores.cpu().numpy(), st.route.scores)
