"""A bounded fuzz of the whole library on the GPU: about a hundred seeded random shapes (batch, group size
including the multi-query groups of 16 and 32, P, K_c, ragged lengths, wide block tables) through every
variant of the step - closed-form weights, both iterative solvers, the routing certificate, group-shared
routing and two-level routing, and 32-token pages - each compared with the CPU oracle exactly as the named tests do (discrete
results bit for bit, floating point within the stated tolerances)."""
import random

import pytest

import test_gpu_certificate as TC
import test_gpu_group_shared as TG
import test_gpu_solver as TS
import test_gpu_two_level as TL
from gpu_runner import compare, run_gpu
from workloads import WorkloadSpec, make_workload

pytestmark = pytest.mark.gpu


def _draw(rng, max_units=600, groups=(1, 2, 4, 8), max_len=3000, wide_p=0.15, max_P=64, max_Kc=700, page=16):
    G = rng.choice(groups)
    hkv = rng.choice([1, 2, 4])
    hq = G * hkv
    batch = rng.randint(1, max(1, max_units // hq))
    P = rng.choice([p for p in (1, 2, 5, 8, 16, 31, 32, 48, 64) if p <= max_P])
    K_c = min(rng.choice([k for k in (1, 7, 40, 100, 256, 300, 700) if k <= max_Kc]), P * page)
    lens = [rng.choice([1, page - 1, page, page + 1, rng.randint(1, 600), rng.randint(1, max_len)]) for _ in range(batch)]
    if rng.random() < wide_p:
        lens[0] = rng.randint(66000, 80000) * (page // 16)     # a block table wider than 4096 pages
    return WorkloadSpec(name="z", config=9, batch=batch, n_q_heads=hq, n_kv_heads=hkv, P=P, K_c=K_c, page_size=page,
                        seq_lens=tuple(lens), needles=rng.choice([0, 1, 3]), needle_positions="uniform")


@pytest.mark.parametrize("seed", range(6))
def test_closed_form_step(seed):
    rng = random.Random(100 + seed)
    for case in range(8):                          # 48 shapes, multi-query groups included
        spec = _draw(rng, groups=(1, 2, 4, 8, 16, 32))
        w = make_workload(spec, seed=20000 + 100 * seed + case)
        compare(w, run_gpu(w), dense_sample=4)


@pytest.mark.parametrize("seed", range(2))
def test_pages_of_32_tokens(seed):
    rng = random.Random(600 + seed)
    for case in range(8):                          # closed-form step, every group size
        spec = _draw(rng, groups=(1, 2, 4, 8, 16, 32), page=32)
        w = make_workload(spec, seed=25000 + 100 * seed + case)
        compare(w, run_gpu(w), dense_sample=4)
    for case in range(4):                          # certificate, two-level routing, one solver each
        spec = _draw(rng, wide_p=0.1, page=32)
        w = make_workload(spec, seed=25500 + 100 * seed + case)
        TC.compare_certified(w, TC.run_certified(w))
        spec = _draw(rng, max_units=300, page=32)
        w = make_workload(spec, seed=25600 + 100 * seed + case)
        P_super = rng.choice([1, 2, 4, 16])
        TL._compare(w, TL._run(w, P_super, spec.P, spec.K_c), P_super, spec.P, spec.K_c)
        spec = _draw(rng, max_units=300, max_len=1500, wide_p=0.0, max_P=16, max_Kc=256, page=32)
        w = make_workload(spec, seed=25700 + 100 * seed + case)
        iters = rng.choice([0, 2, 5])
        TS.compare_entropic(w, TS.run_entropic(w, iters), iters)
        TS.compare_fw(w, TS.run_fw(w, iters), iters)


@pytest.mark.parametrize("kind", ["entropic", "frank_wolfe"])
def test_iterative_solvers(kind):
    rng = random.Random(200 + len(kind))
    for case in range(8):                          # 16 shapes
        spec = _draw(rng, max_units=300, max_len=1500, wide_p=0.0, max_P=16, max_Kc=256)
        w = make_workload(spec, seed=21000 + case)
        iters = rng.choice([0, 2, 5])
        if kind == "entropic":
            TS.compare_entropic(w, TS.run_entropic(w, iters), iters)
        else:
            TS.compare_fw(w, TS.run_fw(w, iters), iters)


def test_routing_certificate():
    rng = random.Random(300)
    for case in range(12):
        spec = _draw(rng, wide_p=0.1)
        w = make_workload(spec, seed=22000 + case)
        TC.compare_certified(w, TC.run_certified(w))


def test_group_shared_routing():
    rng = random.Random(400)
    for case in range(12):
        spec = _draw(rng, max_units=400)
        w = make_workload(spec, seed=23000 + case)
        TG._run_and_compare(w)


def test_two_level_routing():
    rng = random.Random(500)
    for case in range(12):
        spec = _draw(rng, max_units=300)
        w = make_workload(spec, seed=24000 + case)
        P_super = rng.choice([1, 2, 4, 16, 64])
        TL._compare(w, TL._run(w, P_super, spec.P, spec.K_c), P_super, spec.P, spec.K_c)
