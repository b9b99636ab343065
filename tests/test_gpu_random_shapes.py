"""GPU parity on seeded random shapes: batch, group size, P, K_c and ragged lengths drawn so that all
three thread-block shapes of the fused kernel (512, 256 and 128 threads) and both page selections
(registers, shared memory) are reached; same comparisons as the named cases (discrete results bit for
bit against the CPU oracle, floating point within the stated tolerances)."""
import random

import pytest

from gpu_runner import compare, run_gpu
from workloads import WorkloadSpec, make_workload

pytestmark = pytest.mark.gpu


def _draw(rng, lo_units, hi_units, wide):
    hq = rng.choice([4, 8, 16])
    hkv = rng.choice([h for h in (1, 2, 4, 8, 16) if h <= hq and hq % h == 0 and hq // h <= 8])
    batch = rng.randint(max(1, lo_units // hq + 1), max(1, hi_units // hq))
    P = rng.choice([1, 2, 5, 8, 16, 31, 32, 48, 64])
    K_c = min(rng.choice([1, 7, 40, 100, 256, 300, 700]), P * 16)
    lens = [rng.choice([1, 15, 16, 17, rng.randint(1, 600), rng.randint(1, 3000)]) for _ in range(batch)]
    if wide:
        lens[0] = rng.randint(66000, 80000)     # a block table wider than 4096 pages
    return WorkloadSpec(name="r", config=9, batch=batch, n_q_heads=hq, n_kv_heads=hkv, P=P, K_c=K_c,
                        seq_lens=tuple(lens), needles=rng.choice([0, 1, 3]), needle_positions="uniform")


@pytest.mark.parametrize("lo,hi,wide,seed", [
    (0, 148, False, 1), (0, 148, True, 2),          # no more units than SMs: 512 threads
    (148, 296, False, 3), (148, 296, True, 4),      # 256 threads
    (296, 700, False, 5), (296, 700, True, 6),      # 128 threads; wide: selection in shared memory
])
def test_random_shapes(lo, hi, wide, seed):
    rng = random.Random(seed)
    for case in range(4):
        w = make_workload(_draw(rng, lo, hi, wide), seed=9000 + 10 * seed + case)
        compare(w, run_gpu(w), dense_sample=4)
