"""GPU parity of the fp8 (e4m3) KV-cache entry points.  The cache is quantised with one power-of-two scale per
(pool page, KV head) (workloads.quantize_kv_fp8), so every value a byte stands for is exact in bf16 and the
reference is the unchanged oracle run on the bf16 cache that holds those values: summaries, routed pages,
scores, candidate-derived diagnostics, flags and lists bit for bit; outputs within gpu_runner's tolerances."""
import math
import random

import numpy as np
import pytest
import torch

from gpu_runner import GpuRun, compare
from paper_2602_13804_b200 import binding as B
from workloads import WorkloadSpec, make_workload, quantize_kv_fp8

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def spec(**kw):
    base = dict(name="f8", config=9, batch=3, n_q_heads=8, n_kv_heads=2, P=4, K_c=40,
                seq_lens=(700, 333, 45), needles=3, needle_positions="uniform")
    base.update(kw)
    return WorkloadSpec(**base)


def run_fp8(w, gap_threshold=None, alt_strides=False, quantised=None):
    """Returns (the workload whose bf16 caches hold the values of the fp8 cache, the GPU results)."""
    wq, k8, v8, ke, ve = quantised if quantised is not None else quantize_kv_fp8(w)
    P, K_c, eps = w.spec.P, w.spec.K_c, w.epsilon
    tau = w.gap_threshold if gap_threshold is None else gap_threshold
    q, bt, sl = w.q.to(DEV), w.block_table.to(DEV), w.seq_lens.to(DEV)
    k8, v8 = k8.to(DEV), v8.to(DEV)
    if alt_strides:     # cache stored as [pool, page, kv_head, d]
        k8 = k8.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        v8 = v8.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    ks, vs = torch.exp2(ke.float()).to(DEV), torch.exp2(ve.float()).to(DEV)
    shape = B.shape_of(q, k8, bt)
    units = shape.batch * shape.n_q_heads
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries_fp8(shape, k8, ks, bt, sl, None, summ)
    routed = torch.full((shape.batch, shape.n_q_heads, P), -7, dtype=torch.int32, device=DEV)
    rscores = torch.zeros((shape.batch, shape.n_q_heads, P), dtype=torch.float32, device=DEV)
    B.vsa_route_pages(shape, q, summ, bt, sl, P, routed, rscores, B.alloc_workspace(shape, P, K_c, B.VSA_WS_ROUTE, DEV))
    out = torch.full((shape.batch, shape.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    diag = B.alloc_diag(units, DEV)
    flist = torch.full((units,), -1, dtype=torch.int32, device=DEV)
    fcount = torch.full((1,), 12345, dtype=torch.int32, device=DEV)
    B.vsa_sparse_decode_fp8(shape, q, k8, v8, ks, vs, bt, sl, routed, P, K_c, eps, tau, out, diag, flist, fcount)
    out_sparse = out.cpu().numpy().copy()
    diag_sparse = {k: v.numpy() for k, v in B.diag_to_dict(diag).items()}
    B.vsa_dense_decode_fallback_fp8(shape, q, k8, v8, ks, vs, bt, sl, flist, fcount, eps, out, diag,
                                    B.alloc_workspace(shape, P, K_c, B.VSA_WS_DENSE, DEV))
    n = int(fcount.item())
    out2 = torch.full_like(out, float("nan"))
    diag2 = B.alloc_diag(units, DEV)
    routed2 = torch.full_like(routed, -7)
    flist2 = torch.full_like(flist, -1)
    fcount2 = torch.full_like(fcount, 777)
    B.vsa_decode_step_fp8(shape, q, summ, k8, v8, ks, vs, bt, sl, P, K_c, eps, tau, out2, diag2, routed2, flist2, fcount2,
                          B.alloc_workspace(shape, P, K_c, B.VSA_WS_STEP, DEV))
    n2 = int(fcount2.item())
    torch.cuda.synchronize()
    g = GpuRun(summaries=summ, routed_pages=routed.cpu().numpy(), routed_scores=rscores.cpu().numpy(),
               out_sparse=out_sparse, diag_sparse=diag_sparse, out=out.cpu().numpy(),
               diag={k: v.numpy() for k, v in B.diag_to_dict(diag).items()}, fallback_units=np.sort(flist[:n].cpu().numpy()),
               step_out=out2.cpu().numpy(), step_diag={k: v.numpy() for k, v in B.diag_to_dict(diag2).items()},
               step_routed=routed2.cpu().numpy(), step_fallback_units=np.sort(flist2[:n2].cpu().numpy()))
    return wq, g


@pytest.mark.parametrize("hq,hkv", [(8, 2), (8, 1), (4, 4), (2, 1), (16, 1), (32, 2)])
@pytest.mark.parametrize("needles", [3, 0])
def test_small_ragged(hq, hkv, needles):
    w = make_workload(spec(n_q_heads=hq, n_kv_heads=hkv, needles=needles), seed=1100 + hq * 10 + hkv)
    wq, g = run_fp8(w)
    compare(wq, g)


def test_lengths_around_page_and_block_boundaries():
    lens = (16 * 32 * 3 + 5, 16 * 32, 16 * 33 + 15, 1, 15, 16, 17)
    w = make_workload(spec(batch=7, seq_lens=lens, P=8, K_c=100, needles=2), seed=1120)
    compare(*run_fp8(w))


def test_dense_pass_for_every_unit_and_for_none():
    w = make_workload(spec(seq_lens=(2100, 999, 64), needles=0), seed=1130)
    wq, g = run_fp8(w, gap_threshold=math.inf)
    stats = compare(wq, g, gap_threshold=math.inf)
    assert stats["fallback_fraction"] == 1.0
    wq, g = run_fp8(w, gap_threshold=-math.inf)
    compare(wq, g, gap_threshold=-math.inf)


def test_pages_of_32_tokens_and_non_native_strides():
    w = make_workload(spec(page_size=32, seq_lens=(1500, 700, 33), P=3, K_c=64), seed=1140)
    compare(*run_fp8(w))
    wq, g = run_fp8(w, gap_threshold=math.inf)
    compare(wq, g, gap_threshold=math.inf)
    w = make_workload(spec(), seed=1141)
    compare(*run_fp8(w, alt_strides=True))
    wq, g = run_fp8(w, gap_threshold=math.inf, alt_strides=True)
    compare(wq, g, gap_threshold=math.inf)


def test_every_block_size_and_a_wide_table():
    w = make_workload(spec(batch=3, n_q_heads=2, n_kv_heads=1, seq_lens=(5000, 2500, 2049), P=128, K_c=700), seed=1150)
    compare(*run_fp8(w))
    w = make_workload(spec(batch=40, seq_lens=tuple(200 + 37 * i for i in range(40)), P=64, K_c=300, needles=2), seed=1151)
    compare(*run_fp8(w))
    w = make_workload(spec(batch=80, seq_lens=tuple(90 + 21 * i for i in range(80)), P=4, K_c=48, needles=2), seed=1152)
    compare(*run_fp8(w))
    w = make_workload(spec(batch=2, seq_lens=(70000, 900), P=16, K_c=128), seed=1153)
    wq, g = run_fp8(w)
    compare(wq, g, dense_sample=4)


def test_random_shapes():
    rng = random.Random(1160)
    for case in range(12):
        G = rng.choice([1, 2, 4, 8, 16])
        hkv = rng.choice([1, 2, 4])
        hq = G * hkv
        batch = rng.randint(1, max(1, 400 // hq))
        page = rng.choice([16, 32])
        P = rng.choice([p for p in (1, 2, 5, 8, 16, 31, 32, 64) if p * page <= 2048])
        K_c = min(rng.choice([1, 7, 40, 100, 256, 700]), P * page)
        lens = tuple(rng.choice([1, page - 1, page, page + 1, rng.randint(1, 600), rng.randint(1, 3000)]) for _ in range(batch))
        w = make_workload(spec(batch=batch, n_q_heads=hq, n_kv_heads=hkv, P=P, K_c=K_c, page_size=page, seq_lens=lens,
                               needles=rng.choice([0, 1, 3])), seed=27000 + case)
        wq, g = run_fp8(w)
        compare(wq, g, dense_sample=4)


def test_the_quantised_cache_still_finds_the_planted_keys():
    w = make_workload(spec(seq_lens=(4000, 2500, 900), P=8, K_c=64), seed=1170)
    wq, g = run_fp8(w)
    stats = compare(wq, g)
    assert stats["fallback_fraction"] < 0.5


def test_every_byte_value_decodes_exactly_subnormals_included():
    # pages filled with random bytes over the whole e4m3 code space (all but the two NaN codes), so that the
    # subnormal codes 0x01..0x07 / 0x81..0x87 and the largest magnitudes occur in K and V of both passes
    from dataclasses import replace
    w = make_workload(spec(seq_lens=(700, 333, 45), needles=0), seed=1180)
    wq, k8, v8, ke, ve = quantize_kv_fp8(w)
    gen = torch.Generator().manual_seed(7)
    codes = torch.tensor([b for b in range(256) if (b & 0x7f) != 0x7f], dtype=torch.uint8)
    k8 = codes[torch.randint(0, len(codes), k8.shape, generator=gen)]
    v8 = codes[torch.randint(0, len(codes), v8.shape, generator=gen)]
    ke = torch.randint(-12, -6, ke.shape, generator=gen).to(torch.int8)     # scores of a few units, not thousands
    ve = torch.randint(-12, -8, ve.shape, generator=gen).to(torch.int8)     # values of order one

    def deq(raw, ex):
        return (raw.view(torch.float8_e4m3fn).float() * torch.exp2(ex.float())[:, :, None, None]).to(torch.bfloat16)
    kd, vd = deq(k8, ke), deq(v8, ve)
    assert torch.equal(kd.float(), k8.view(torch.float8_e4m3fn).float() * torch.exp2(ke.float())[:, :, None, None])
    wq = replace(wq, k_cache=kd, v_cache=vd)
    for tau in (w.gap_threshold, math.inf):
        wq2, g = run_fp8(w, gap_threshold=tau, quantised=(wq, k8, v8, ke, ve))
        compare(wq2, g, gap_threshold=tau)


def test_subnormal_codes_are_not_flushed_in_either_pass():
    # a cache made of e4m3 subnormal codes only (m * 2^-9, m = 0..7, both signs) with scale 2^9: the values are
    # the integers -7..7, so a decode that flushed subnormals to zero would give uniform weights and zero output
    from dataclasses import replace
    w = make_workload(spec(seq_lens=(300, 177, 45), needles=0, epsilon=8.0), seed=1190)
    wq, k8, v8, ke, ve = quantize_kv_fp8(w)
    gen = torch.Generator().manual_seed(9)
    codes = torch.tensor(list(range(0, 8)) + list(range(0x80, 0x88)), dtype=torch.uint8)
    k8 = codes[torch.randint(0, 16, k8.shape, generator=gen)]
    v8 = codes[torch.randint(0, 16, v8.shape, generator=gen)]
    ke = torch.full_like(ke, 9)
    ve = torch.full_like(ve, 9)
    kd = (k8.view(torch.float8_e4m3fn).float() * 512.0).to(torch.bfloat16)
    vd = (v8.view(torch.float8_e4m3fn).float() * 512.0).to(torch.bfloat16)
    assert set(kd.float().unique().tolist()) <= set(float(i) for i in range(-7, 8)) and kd.float().abs().max() == 7.0
    wq = replace(wq, k_cache=kd, v_cache=vd)
    for tau in (-math.inf, math.inf):
        wq2, g = run_fp8(w, gap_threshold=tau, quantised=(wq, k8, v8, ke, ve))
        compare(wq2, g, gap_threshold=tau)
        assert np.abs(g.out).max() > 0.5     # the readout is far from zero
