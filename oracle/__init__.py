"""CPU oracle (test infrastructure only).

Thin numpy/ctypes front end of ``vsa_oracle.c``.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library never does, and this
package never imports the CUDA library.

All array arguments are host numpy arrays.  bf16 tensors are passed as ``uint16`` bit
patterns (``torch_tensor.view(torch.int16).numpy().view(np.uint16)``).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vsa_oracle.c")
_LIB = os.path.join(_HERE, "libvsa_oracle.so")
_CFLAGS = ["-O2", "-fopenmp", "-ffp-contract=off", "-std=c99", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Shape(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32),
        ("num_pool_pages", C.c_int64),
        ("kv_page_stride", C.c_int64), ("kv_head_stride", C.c_int64), ("kv_token_stride", C.c_int64),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_canon_dot.restype = C.c_float
        _lib.orc_canon_dot_d.restype = C.c_float
        _lib.orc_bf16_to_f32.restype = C.c_float
        _lib.orc_f32_to_bf16.restype = C.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [C.c_float]
        _lib.orc_bf16_to_f32.argtypes = [C.c_uint16]
        _lib.orc_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def set_num_threads(n: int) -> None:
    lib().orc_set_num_threads(C.c_int(int(n)))


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, f"bf16 data must be passed as uint16 bit patterns, got {a.dtype}"
    return a


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


@dataclass
class Geometry:
    """Shape of a paged cache: K/V pools are [pool, n_kv, page, d] unless strides say otherwise."""
    batch: int
    n_q_heads: int
    n_kv_heads: int
    max_pages_per_seq: int
    num_pool_pages: int
    head_dim: int = 128
    page_size: int = 16
    kv_page_stride: Optional[int] = None
    kv_head_stride: Optional[int] = None
    kv_token_stride: Optional[int] = None

    def c(self) -> _Shape:
        ts = self.kv_token_stride or self.head_dim
        hs = self.kv_head_stride or self.page_size * ts
        ps = self.kv_page_stride or self.n_kv_heads * hs
        return _Shape(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.page_size,
                      self.max_pages_per_seq, self.num_pool_pages, ps, hs, ts)

    @property
    def units(self) -> int:
        return self.batch * self.n_q_heads


def bf16_to_f32(bits) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16(x) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    f = lib().orc_f32_to_bf16
    flat_in, flat_out = x.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = f(C.c_float(float(flat_in[i])))
    return out


def canon_dot(x_bits, y_bits) -> np.float32:
    x, y = _u16(x_bits), _u16(y_bits)
    assert x.size == y.size and x.size in (64, 128, 256)
    return np.float32(lib().orc_canon_dot_d(_p(x), _p(y), C.c_int(int(x.size))))


def build_summaries(geo: Geometry, k_cache, block_table, seq_lens, first_page=None,
                    summaries: Optional[np.ndarray] = None) -> np.ndarray:
    k = _u16(k_cache)
    bt, sl = _i32(block_table), _i32(seq_lens)
    if summaries is None:
        summaries = np.zeros((geo.num_pool_pages, geo.n_kv_heads, geo.head_dim), dtype=np.uint16)
    fp = None if first_page is None else _i32(first_page)
    s = geo.c()
    rc = lib().orc_build_summaries(C.byref(s), _p(k), _p(bt), _p(sl), _p(fp), _p(summaries))
    assert rc == 0, rc
    return summaries


@dataclass
class RouteResult:
    pages: np.ndarray       # int32 [B, Hq, P], -1 padded, in (score desc, page asc) order
    scores: np.ndarray      # fp32 [B, Hq, P]
    all_scores: Optional[np.ndarray]  # fp32 [B, Hq, max_pages] (entries past n_b undefined)


def route(geo: Geometry, q, summaries, block_table, seq_lens, P: int, want_all_scores=False) -> RouteResult:
    qb, sm = _u16(q), _u16(summaries)
    bt, sl = _i32(block_table), _i32(seq_lens)
    pages = np.empty((geo.batch, geo.n_q_heads, P), dtype=np.int32)
    scores = np.empty((geo.batch, geo.n_q_heads, P), dtype=np.float32)
    alls = np.full((geo.batch, geo.n_q_heads, geo.max_pages_per_seq), -np.inf, dtype=np.float32) \
        if want_all_scores else None
    s = geo.c()
    rc = lib().orc_route(C.byref(s), _p(qb), _p(sm), _p(bt), _p(sl), C.c_int(P), _p(pages), _p(scores), _p(alls))
    assert rc == 0, rc
    return RouteResult(pages, scores, alls)


SUPER = 16    # logical pages per super-page


def n_supers(max_pages_per_seq: int) -> int:
    return (max_pages_per_seq + SUPER - 1) // SUPER


def build_super_summaries(geo: Geometry, summaries, block_table, seq_lens):
    """(super_summaries uint16 [B, max_supers, Hkv, d], super_rep int32 [B, max_supers, Hkv]): per
    super-page of 16 logical pages the page summary of largest fp32 squared norm (ties: lowest page)."""
    sm = _u16(summaries)
    bt, sl = _i32(block_table), _i32(seq_lens)
    ms = n_supers(geo.max_pages_per_seq)
    sup = np.zeros((geo.batch, ms, geo.n_kv_heads, geo.head_dim), np.uint16)
    rep = np.full((geo.batch, ms, geo.n_kv_heads), -1, np.int32)
    s = geo.c()
    rc = lib().orc_build_super_summaries(C.byref(s), _p(sm), _p(bt), _p(sl), C.c_int(ms), _p(sup), _p(rep))
    assert rc == 0, rc
    return sup, rep


@dataclass
class TwoLevelRouteResult:
    supers: np.ndarray      # int32 [B, Hq, P_super] super-pages kept, (score desc, index asc), -1 padded
    pages: np.ndarray       # int32 [B, Hq, P]
    scores: np.ndarray      # fp32 [B, Hq, P]


def route_two_level(geo: Geometry, q, summaries, super_summaries, block_table, seq_lens, P_super: int,
                    P: int) -> TwoLevelRouteResult:
    qb, sm, sup = _u16(q), _u16(summaries), _u16(super_summaries)
    bt, sl = _i32(block_table), _i32(seq_lens)
    supers = np.empty((geo.batch, geo.n_q_heads, P_super), np.int32)
    pages = np.empty((geo.batch, geo.n_q_heads, P), np.int32)
    scores = np.empty((geo.batch, geo.n_q_heads, P), np.float32)
    s = geo.c()
    rc = lib().orc_route_two_level(C.byref(s), _p(qb), _p(sm), _p(sup), C.c_int(sup.shape[1]), _p(bt), _p(sl),
                                   C.c_int(P_super), C.c_int(P), _p(supers), _p(pages), _p(scores))
    assert rc == 0, rc
    return TwoLevelRouteResult(supers, pages, scores)


@dataclass
class SparseResult:
    out: np.ndarray           # fp64 [B, Hq, d]
    delta: np.ndarray         # fp32 [B, Hq]  s(1) - best rejected scored token (+inf if none)
    delta12: np.ndarray       # fp32 [B, Hq]  s(1) - s(2)
    s_max: np.ndarray         # fp32 [B, Hq]
    lse: np.ndarray           # fp64 [B, Hq]
    leak_bound: np.ndarray    # fp64 [B, Hq]
    n_candidates: np.ndarray  # int32 [B, Hq]
    fallback: np.ndarray      # int32 [B, Hq]
    cand_pos: np.ndarray      # int32 [B, Hq, K_c] token positions, -1 padded, selection order
    cand_weight: np.ndarray   # fp64 [B, Hq, K_c] normalised weights
    best_rejected: np.ndarray = None   # fp32 [B, Hq] best scored token outside S, -inf if none


def sparse(geo: Geometry, q, k_cache, v_cache, block_table, seq_lens, routed_pages, K_c: int,
           epsilon: float, gap_threshold: float) -> SparseResult:
    qb, k, v = _u16(q), _u16(k_cache), _u16(v_cache)
    bt, sl, rp = _i32(block_table), _i32(seq_lens), _i32(routed_pages)
    B, H, d = geo.batch, geo.n_q_heads, geo.head_dim
    P = rp.shape[-1]
    r = SparseResult(
        out=np.zeros((B, H, d)), delta=np.zeros((B, H), np.float32), delta12=np.zeros((B, H), np.float32),
        s_max=np.zeros((B, H), np.float32), lse=np.zeros((B, H)), leak_bound=np.zeros((B, H)),
        n_candidates=np.zeros((B, H), np.int32), fallback=np.zeros((B, H), np.int32),
        cand_pos=np.full((B, H, K_c), -1, np.int32), cand_weight=np.zeros((B, H, K_c)),
        best_rejected=np.zeros((B, H), np.float32))
    s = geo.c()
    rc = lib().orc_sparse(C.byref(s), _p(qb), _p(k), _p(v), _p(bt), _p(sl), _p(rp), C.c_int(P), C.c_int(K_c),
                          C.c_float(epsilon), C.c_float(gap_threshold), _p(r.out), _p(r.delta), _p(r.delta12),
                          _p(r.s_max), _p(r.lse), _p(r.leak_bound), _p(r.n_candidates), _p(r.fallback),
                          _p(r.cand_pos), _p(r.cand_weight), _p(r.best_rejected))
    assert rc == 0, rc
    return r


def route_group(geo: Geometry, q, summaries, block_table, seq_lens, P: int) -> RouteResult:
    """Group-shared page routing: pages int32 [B, Hkv, P], scores fp32 [B, Hkv, P] (summed over the group)."""
    qb, sm = _u16(q), _u16(summaries)
    bt, sl = _i32(block_table), _i32(seq_lens)
    pages = np.empty((geo.batch, geo.n_kv_heads, P), dtype=np.int32)
    scores = np.empty((geo.batch, geo.n_kv_heads, P), dtype=np.float32)
    s = geo.c()
    rc = lib().orc_route_group(C.byref(s), _p(qb), _p(sm), _p(bt), _p(sl), C.c_int(P), _p(pages), _p(scores))
    assert rc == 0, rc
    return RouteResult(pages, scores, None)


def sparse_group(geo: Geometry, q, k_cache, v_cache, block_table, seq_lens, routed_pages, K_c: int,
                 epsilon: float, gap_threshold: float) -> SparseResult:
    """Group-shared candidates: routed_pages [B, Hkv, P]; per-unit outputs and diagnostics; cand_pos is
    [B, Hkv, K_c] (one candidate set per KV head).  cand_weight / best_rejected are not filled."""
    qb, k, v = _u16(q), _u16(k_cache), _u16(v_cache)
    bt, sl, rp = _i32(block_table), _i32(seq_lens), _i32(routed_pages)
    B, H, d = geo.batch, geo.n_q_heads, geo.head_dim
    P = rp.shape[-1]
    r = SparseResult(
        out=np.zeros((B, H, d)), delta=np.zeros((B, H), np.float32), delta12=np.zeros((B, H), np.float32),
        s_max=np.zeros((B, H), np.float32), lse=np.zeros((B, H)), leak_bound=np.zeros((B, H)),
        n_candidates=np.zeros((B, H), np.int32), fallback=np.zeros((B, H), np.int32),
        cand_pos=np.full((B, geo.n_kv_heads, K_c), -1, np.int32), cand_weight=None, best_rejected=None)
    s = geo.c()
    rc = lib().orc_sparse_group(C.byref(s), _p(qb), _p(k), _p(v), _p(bt), _p(sl), _p(rp), C.c_int(P), C.c_int(K_c),
                                C.c_float(epsilon), C.c_float(gap_threshold), _p(r.out), _p(r.delta), _p(r.delta12),
                                _p(r.s_max), _p(r.lse), _p(r.leak_bound), _p(r.n_candidates), _p(r.fallback),
                                _p(r.cand_pos))
    assert rc == 0, rc
    return r


def build_radii(geo: Geometry, k_cache, summaries, block_table, seq_lens, first_page=None, radii=None) -> np.ndarray:
    """fp32 [pool, Hkv]: the slack-inflated radius of every owned page around its stored summary."""
    k, sm = _u16(k_cache), _u16(summaries)
    bt, sl = _i32(block_table), _i32(seq_lens)
    if radii is None:
        radii = np.zeros((geo.num_pool_pages, geo.n_kv_heads), np.float32)
    fp = None if first_page is None else _i32(first_page)
    s = geo.c()
    rc = lib().orc_build_radii(C.byref(s), _p(k), _p(sm), _p(bt), _p(sl), _p(fp), _p(radii))
    assert rc == 0, rc
    return radii


@dataclass
class CertResult:
    ub_unrouted: np.ndarray   # fp32 [B, Hq]
    delta_cert: np.ndarray    # fp32 [B, Hq]
    certified: np.ndarray     # int32 [B, Hq]
    leak_cert: np.ndarray     # fp64 [B, Hq]


def certify(geo: Geometry, q, radii, block_table, seq_lens, route: "RouteResult", sp: SparseResult,
            epsilon: float, gap_threshold: float) -> CertResult:
    """Certified gap of every unit from the page scores of `route` (made with want_all_scores=True)
    and the closed-form pass `sp`."""
    assert route.all_scores is not None
    qb, bt, sl = _u16(q), _i32(block_table), _i32(seq_lens)
    B, H = geo.batch, geo.n_q_heads
    rp = _i32(route.pages)
    r = CertResult(np.zeros((B, H), np.float32), np.zeros((B, H), np.float32), np.zeros((B, H), np.int32),
                   np.zeros((B, H)))
    rad = np.ascontiguousarray(radii, dtype=np.float32)
    alls = np.ascontiguousarray(route.all_scores, dtype=np.float32)
    s = geo.c()
    rc = lib().orc_certify(C.byref(s), _p(qb), _p(rad), _p(bt), _p(sl), _p(alls), _p(rp), C.c_int(rp.shape[-1]),
                           _p(np.ascontiguousarray(sp.s_max)), _p(np.ascontiguousarray(sp.best_rejected)),
                           _p(np.ascontiguousarray(sp.n_candidates)), C.c_float(epsilon), C.c_float(gap_threshold),
                           _p(r.ub_unrouted), _p(r.delta_cert), _p(r.certified), _p(r.leak_cert))
    assert rc == 0, rc
    return r


@dataclass
class FrankWolfeResult:
    alpha: np.ndarray       # fp32 [B, Hq, K_c] weights in the order of cand_pos
    fw_gap: np.ndarray      # fp32 [B, Hq]
    objective: np.ndarray   # fp32 [B, Hq]  1/2 |K_S^T a - q|^2
    residual2: np.ndarray
    step: np.ndarray        # last gamma


def frank_wolfe(geo: Geometry, q, k_cache, block_table, cand_pos, iters: int) -> FrankWolfeResult:
    qb, k, bt = _u16(q), _u16(k_cache), _i32(block_table)
    cp = _i32(cand_pos)
    B, H, K_c = geo.batch, geo.n_q_heads, cp.shape[-1]
    r = FrankWolfeResult(np.zeros((B, H, K_c), np.float32), np.zeros((B, H), np.float32), np.zeros((B, H), np.float32),
                         np.zeros((B, H), np.float32), np.zeros((B, H), np.float32))
    s = geo.c()
    rc = lib().orc_frank_wolfe(C.byref(s), _p(qb), _p(k), _p(bt), _p(cp), C.c_int(K_c), C.c_int(iters), _p(r.alpha),
                               _p(r.fw_gap), _p(r.objective), _p(r.residual2), _p(r.step))
    assert rc == 0, rc
    return r


@dataclass
class DenseResult:
    out: np.ndarray                    # fp64 [B, Hq, d] (rows of unmasked units only)
    lse: np.ndarray                    # fp64 [B, Hq]
    true_leak: Optional[np.ndarray]    # dense softmax mass outside the candidate set
    true_gap: Optional[np.ndarray]     # max_t s_t - max_{j not in S} s_j
    y_off: Optional[np.ndarray]        # dense readout restricted to the complement of S


def dense(geo: Geometry, q, k_cache, v_cache, block_table, seq_lens, epsilon: float,
          unit_mask=None, cand_pos=None) -> DenseResult:
    qb, k, v = _u16(q), _u16(k_cache), _u16(v_cache)
    bt, sl = _i32(block_table), _i32(seq_lens)
    B, H, d = geo.batch, geo.n_q_heads, geo.head_dim
    out, lse = np.zeros((B, H, d)), np.zeros((B, H))
    um = None if unit_mask is None else _i32(unit_mask)
    cp = leak = gap = yoff = None
    K_c = 0
    if cand_pos is not None:
        cp = _i32(cand_pos)
        K_c = cp.shape[-1]
        leak, gap, yoff = np.zeros((B, H)), np.zeros((B, H)), np.zeros((B, H, d))
    s = geo.c()
    rc = lib().orc_dense(C.byref(s), _p(qb), _p(k), _p(v), _p(bt), _p(sl), C.c_float(epsilon), _p(um),
                         _p(out), _p(lse), _p(cp), C.c_int(K_c), _p(leak), _p(gap), _p(yoff))
    assert rc == 0, rc
    return DenseResult(out, lse, leak, gap, yoff)


@dataclass
class StepResult:
    summaries: np.ndarray
    route: RouteResult
    sparse: SparseResult
    out: np.ndarray     # fp64 [B, Hq, d]: sparse output, dense output where fallback = 1
    lse: np.ndarray
    dense: Optional[DenseResult]


def decode_step(geo: Geometry, q, k_cache, v_cache, block_table, seq_lens, P: int, K_c: int,
                epsilon: float, gap_threshold: float, summaries=None) -> StepResult:
    """Whole step in the paper's order: summaries (if not given) -> page routing -> token
    routing + candidate softmax + diagnostics -> dense attention for the flagged units."""
    if summaries is None:
        summaries = build_summaries(geo, k_cache, block_table, seq_lens)
    r = route(geo, q, summaries, block_table, seq_lens, P)
    sp = sparse(geo, q, k_cache, v_cache, block_table, seq_lens, r.pages, K_c, epsilon, gap_threshold)
    out, lse = sp.out.copy(), sp.lse.copy()
    dn = None
    if sp.fallback.any():
        dn = dense(geo, q, k_cache, v_cache, block_table, seq_lens, epsilon, unit_mask=sp.fallback)
        flagged = sp.fallback.astype(bool)
        out[flagged] = dn.out[flagged]
        lse[flagged] = dn.lse[flagged]
    return StepResult(summaries, r, sp, out, lse, dn)
