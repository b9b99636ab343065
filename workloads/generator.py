"""Seeded generator for paged-KV decode workloads.

Recipe (identical for every configuration):

* ``q``, K and V are iid N(0, 1) drawn in fp32 and rounded to bf16 (RNE).
* "Needles" give the cache retrieval structure: for KV head ``g`` of sequence
  ``b`` the needle key is ``bf16(4 * q_hat + 0.1 * N(0, I))`` where ``q_hat``
  is the sum of the query vectors of the heads that read KV head ``g``
  (``needle_mode="group_sum"``), a single head of the group chosen round-robin
  (``"per_qhead_round_robin"``) or the first head's unit vector
  (``"unit_literal"``).  Values are never touched.
* Physical pages are the prefix of a seeded permutation of the pool, so the
  block tables are random and sequences never share a page.
* Layout: ``k_cache``/``v_cache`` are ``[pool_pages, n_kv_heads, page_size,
  head_dim]`` bf16, ``block_table`` is ``[batch, max_pages_per_seq]`` int32
  (unused entries are -1), ``seq_lens`` is ``[batch]`` int32.

Nothing here computes a page summary, a score or a softmax.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List, Optional, Sequence, Tuple, Union

import torch

HEAD_DIM = 128
PAGE_SIZE = 16
SEED_BASE = 0x5EED0000


def seed_for(config: int, sub: int = 0, rep: int = 0) -> int:
    """Seed of one generated cache: base + 1000*config + 10*sub + rep."""
    return SEED_BASE + 1000 * int(config) + 10 * int(sub) + int(rep)


@dataclass(frozen=True)
class WorkloadSpec:
    name: str
    config: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    P: int
    K_c: int
    # context lengths: a single T for every sequence, explicit per-sequence
    # lengths, or a (lo, hi) range drawn log-uniformly per sequence
    T: Optional[int] = None
    seq_lens: Optional[Tuple[int, ...]] = None
    ragged_T: Optional[Tuple[int, int]] = None
    # needles per (sequence, kv head): a count, or an inclusive (lo, hi) range
    needles: Union[int, Tuple[int, int]] = 0
    # how many sequences get needles (None = all); chosen by seeded permutation
    needle_seqs: Optional[int] = None
    needle_positions: str = "stratified"          # or "uniform"
    needle_mode: str = "group_sum"
    pool_pages: Optional[int] = None               # None = pow2 >= 1.25 * used
    head_dim: int = HEAD_DIM
    page_size: int = PAGE_SIZE
    epsilon: float = math.sqrt(128.0)              # temperature on raw dots
    gap_threshold_in_eps: float = 8.0              # tau = 8 * epsilon
    layers: int = 1

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


@dataclass
class Workload:
    spec: WorkloadSpec
    seed: int
    q: torch.Tensor            # bf16 [B, Hq, d]
    k_cache: torch.Tensor      # bf16 [pool, Hkv, page, d]
    v_cache: torch.Tensor      # bf16 [pool, Hkv, page, d]
    block_table: torch.Tensor  # int32 [B, max_pages]
    seq_lens: torch.Tensor     # int32 [B]
    epsilon: float             # fp32-representable
    gap_threshold: float       # fp32-representable
    needle_positions: List[List[List[int]]] = field(default_factory=list)
    needle_seq_ids: List[int] = field(default_factory=list)

    @property
    def pool_pages(self) -> int:
        return int(self.k_cache.shape[0])

    @property
    def max_pages_per_seq(self) -> int:
        return int(self.block_table.shape[1])

    def to(self, device) -> "Workload":
        return replace(
            self,
            q=self.q.to(device),
            k_cache=self.k_cache.to(device),
            v_cache=self.v_cache.to(device),
            block_table=self.block_table.to(device),
            seq_lens=self.seq_lens.to(device),
        )


CONFIGS = {
    # single decode step, planted needles at uniform positions
    0: WorkloadSpec(name="cfg0_b1_t4k", config=0, batch=1, n_q_heads=32, n_kv_heads=8,
                    T=4096, needles=8, needle_positions="uniform", P=16, K_c=128),
    # Llama-3-8B attention shape, batch 8, 32k context, 64k-page pool, x32 layers
    1: WorkloadSpec(name="cfg1_b8_t32k", config=1, batch=8, n_q_heads=32, n_kv_heads=8,
                    T=32768, needles=32, P=32, K_c=256, pool_pages=65536, layers=32),
    # context sweep point (override batch / T through config_spec)
    2: WorkloadSpec(name="cfg2_sweep", config=2, batch=1, n_q_heads=32, n_kv_heads=8,
                    T=4096, needles=32, P=32, K_c=256),
    # small-gap regime: iid keys, needles only in 4 of the 16 sequences
    3: WorkloadSpec(name="cfg3_fallback", config=3, batch=16, n_q_heads=32, n_kv_heads=8,
                    T=65536, needles=32, needle_seqs=4, P=32, K_c=256),
    # ragged serving batch, GQA 8:1
    4: WorkloadSpec(name="cfg4_ragged", config=4, batch=64, n_q_heads=64, n_kv_heads=8,
                    ragged_T=(4096, 131072), needles=(4, 64), P=64, K_c=512),
}


def config_spec(config: int, **overrides) -> WorkloadSpec:
    """A named configuration, optionally with fields overridden (sweeps, shrunk tests)."""
    spec = CONFIGS[config]
    if overrides:
        spec = replace(spec, **overrides)
        if "name" not in overrides:
            tag = "_".join(f"{k}{v}" for k, v in sorted(overrides.items())
                           if k in ("batch", "T", "P", "K_c"))
            spec = replace(spec, name=f"{spec.name}[{tag}]")
    return spec


def _f32(x: float) -> float:
    return float(torch.tensor(x, dtype=torch.float32).item())


def _draw_seq_lens(spec: WorkloadSpec, gen: torch.Generator) -> List[int]:
    if spec.seq_lens is not None:
        assert len(spec.seq_lens) == spec.batch
        return [int(t) for t in spec.seq_lens]
    if spec.ragged_T is not None:
        lo, hi = spec.ragged_T
        u = torch.rand(spec.batch, generator=gen, dtype=torch.float64)
        ln = math.log(lo) + u * (math.log(hi) - math.log(lo))
        return [max(1, int(math.floor(math.exp(v)))) for v in ln.tolist()]
    assert spec.T is not None
    return [int(spec.T)] * spec.batch


def _needle_positions(T: int, n: int, mode: str, gen: torch.Generator) -> List[int]:
    n = min(n, T)
    if n <= 0:
        return []
    if mode == "uniform":
        return sorted(torch.randperm(T, generator=gen)[:n].tolist())
    if mode == "stratified":
        out = []
        for i in range(n):
            lo = (i * T) // n
            hi = ((i + 1) * T) // n
            off = int(torch.randint(0, max(1, hi - lo), (1,), generator=gen).item())
            out.append(min(T - 1, lo + off))
        return out
    raise ValueError(f"unknown needle position mode {mode!r}")


def make_workload(spec: WorkloadSpec, seed: Optional[int] = None, device="cpu",
                  sub: int = 0, rep: int = 0) -> Workload:
    """Draw one cache + query batch.

    Host-side structure (lengths, block tables, needle positions) always comes
    from a CPU generator seeded with ``seed`` (default: ``seed_for(config, sub)``);
    the large tensors are drawn on ``device`` with a generator of that device
    seeded with ``seed + 1 + rep``, so ``rep`` selects one of several caches with
    identical structure and different contents (the layers of one model).
    """
    # `rep` (the layer-cache index) changes the contents only: all layer caches of one workload share
    # the sequence lengths, block tables and needle positions, as the layers of one model do
    if seed is None:
        seed = seed_for(spec.config, sub, 0)
    device = torch.device(device)
    hgen = torch.Generator(device="cpu").manual_seed(seed)
    dgen = torch.Generator(device=device).manual_seed(seed + 1 + int(rep))
    seed = seed + int(rep)

    B, Hq, Hkv, d, bs = spec.batch, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.page_size
    assert Hq % Hkv == 0
    G = Hq // Hkv

    seq_lens = _draw_seq_lens(spec, hgen)
    n_pages = [(t + bs - 1) // bs for t in seq_lens]
    used = sum(n_pages)
    max_pages = max(n_pages)
    if spec.pool_pages is not None:
        pool = int(spec.pool_pages)
    else:
        pool = 1
        while pool < math.ceil(1.25 * used):
            pool *= 2
    assert pool >= used, "pool too small for the requested sequences"

    perm = torch.randperm(pool, generator=hgen)[:used].to(torch.int32)
    block_table = torch.full((B, max_pages), -1, dtype=torch.int32)
    o = 0
    for b in range(B):
        block_table[b, : n_pages[b]] = perm[o:o + n_pages[b]]
        o += n_pages[b]

    # which sequences get needles, how many per (sequence, kv head), and where
    if spec.needle_seqs is None:
        needle_seq_ids = list(range(B))
    else:
        needle_seq_ids = sorted(torch.randperm(B, generator=hgen)[: spec.needle_seqs].tolist())
    positions: List[List[List[int]]] = [[[] for _ in range(Hkv)] for _ in range(B)]
    for b in needle_seq_ids:
        for g in range(Hkv):
            if isinstance(spec.needles, tuple):
                lo, hi = spec.needles
                n = int(torch.randint(lo, hi + 1, (1,), generator=hgen).item())
            else:
                n = int(spec.needles)
            positions[b][g] = _needle_positions(seq_lens[b], n, spec.needle_positions, hgen)

    # queries
    q = torch.randn((B, Hq, d), generator=dgen, device=device, dtype=torch.float32).to(torch.bfloat16)

    # pools: only pages that some sequence owns are random, the rest stay zero
    k_cache = torch.zeros((pool, Hkv, bs, d), dtype=torch.bfloat16, device=device)
    v_cache = torch.zeros((pool, Hkv, bs, d), dtype=torch.bfloat16, device=device)
    used_ids = perm.to(device=device, dtype=torch.long)
    chunk = 2048
    for s in range(0, used, chunk):
        ids = used_ids[s:s + chunk]
        shape = (ids.numel(), Hkv, bs, d)
        k_cache[ids] = torch.randn(shape, generator=dgen, device=device, dtype=torch.float32).to(torch.bfloat16)
        v_cache[ids] = torch.randn(shape, generator=dgen, device=device, dtype=torch.float32).to(torch.bfloat16)

    # needles overwrite K rows (V untouched)
    rows_b, rows_g, rows_pos, rows_n = [], [], [], []
    for b in needle_seq_ids:
        for g in range(Hkv):
            for i, p in enumerate(positions[b][g]):
                rows_b.append(b); rows_g.append(g); rows_pos.append(p); rows_n.append(i)
    if rows_b:
        tb = torch.tensor(rows_b, device=device, dtype=torch.long)
        tg = torch.tensor(rows_g, device=device, dtype=torch.long)
        tp = torch.tensor(rows_pos, device=device, dtype=torch.long)
        tn = torch.tensor(rows_n, device=device, dtype=torch.long)
        qf = q.to(torch.float32).view(B, Hkv, G, d)
        if spec.needle_mode == "group_sum":
            q_hat = qf.sum(dim=2)[tb, tg]
        elif spec.needle_mode == "per_qhead_round_robin":
            q_hat = qf[tb, tg, tn % G]
        elif spec.needle_mode == "unit_literal":
            v = qf[tb, tg, 0]
            q_hat = v / v.norm(dim=-1, keepdim=True)
        else:
            raise ValueError(f"unknown needle mode {spec.needle_mode!r}")
        noise = torch.randn((len(rows_b), d), generator=dgen, device=device, dtype=torch.float32)
        rows = (4.0 * q_hat + 0.1 * noise).to(torch.bfloat16)
        phys = block_table.to(device)[tb, tp // bs].to(torch.long)
        k_cache[phys, tg, tp % bs] = rows

    eps = _f32(spec.epsilon)
    tau = _f32(spec.gap_threshold_in_eps * eps)
    return Workload(
        spec=spec, seed=seed, q=q, k_cache=k_cache, v_cache=v_cache,
        block_table=block_table.to(device),
        seq_lens=torch.tensor(seq_lens, dtype=torch.int32, device=device),
        epsilon=eps, gap_threshold=tau,
        needle_positions=positions, needle_seq_ids=needle_seq_ids,
    )


def quantize_kv_fp8(w: Workload):
    """An fp8 copy of a workload's KV cache: e4m3 values with one power-of-two scale per (pool page, KV head).

    For every (page, KV head) block of K (and of V) the exponent e is the smallest integer with
    max|x| / 2^e <= 448 (the largest e4m3 value), the stored byte is round-to-nearest-even e4m3 of x / 2^e,
    and the value it stands for is byte * 2^e.  Because the scale is a power of two, that value is exactly
    representable in bf16, so the returned workload - whose bf16 caches hold exactly the values the fp8 cache
    stands for - is what a reference for the fp8 path computes on.

    Returns (workload with the dequantised bf16 caches, k8, v8, k_exp, v_exp): uint8 [pool, Hkv, page, d]
    and int8 [pool, Hkv].
    """
    out = []
    for x in (w.k_cache, w.v_cache):
        xf = x.to(torch.float32)
        amax = xf.abs().amax(dim=(2, 3))                                   # [pool, Hkv]
        e = torch.ceil(torch.log2(torch.clamp(amax, min=1e-30) / 448.0))
        e = torch.where(amax > 0, e, torch.zeros_like(e)).clamp(-100, 100)
        # log2 can land one ulp low at exact powers of two: make sure the scaled block fits
        e = torch.where(amax / torch.exp2(e) > 448.0, e + 1, e)
        scale = torch.exp2(e)[:, :, None, None]
        q8 = (xf / scale).to(torch.float8_e4m3fn)
        deq = (q8.to(torch.float32) * scale).to(torch.bfloat16)
        assert torch.equal(deq.to(torch.float32), q8.to(torch.float32) * scale)   # exact in bf16
        out.append((q8.view(torch.uint8), e.to(torch.int8), deq))
    (k8, ke, kd), (v8, ve, vd) = out
    from dataclasses import replace as _replace
    return _replace(w, k_cache=kd, v_cache=vd), k8, v8, ke, ve
