"""ctypes binding of libvsa.so: argument marshalling only.

Every function has the name and argument order of its C entry point (include/vsa.h) and takes
torch tensors where C takes pointers.  Tensors are used for their device memory and nothing
else: no step of the decode path runs in PyTorch.  The library must be present - there is no
fallback; a missing or unloadable libvsa.so raises at import of this module's ``lib()``.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvsa.so")

VSA_WS_ROUTE, VSA_WS_SPARSE, VSA_WS_DENSE, VSA_WS_STEP, VSA_WS_STEP_CERTIFIED, VSA_WS_STEP_EXPAND = 1, 2, 3, 4, 5, 6
VSA_WS_ROUTE_TWO_LEVEL, VSA_WS_STEP_TWO_LEVEL = 7, 8
VSA_SUPER_PAGES = 16
DIAG_BYTES = 32
DIAG_FIELDS = ("delta", "delta12", "s_max", "lse", "leak_bound", "n_candidates", "fallback", "status")


class VsaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where} failed: {lib().vsa_strerror(code).decode()} ({code})")


class vsa_shape_t(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32),
        ("num_pool_pages", C.c_int64),
        ("kv_page_stride", C.c_int64), ("kv_head_stride", C.c_int64), ("kv_token_stride", C.c_int64),
    ]


class vsa_diag_t(C.Structure):
    _fields_ = [
        ("delta", C.c_float), ("delta12", C.c_float), ("s_max", C.c_float), ("lse", C.c_float),
        ("leak_bound", C.c_float), ("n_candidates", C.c_int32), ("fallback", C.c_int32), ("status", C.c_int32),
    ]


assert C.sizeof(vsa_diag_t) == DIAG_BYTES

_lib = None


def lib() -> C.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (python -m paper_2602_13804_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_13804_b200.build`; "
                               "there is no fallback path")
        _lib = C.CDLL(LIB_PATH)
        vp, i32, f32, sz = C.c_void_p, C.c_int32, C.c_float, C.c_size_t
        shp = C.POINTER(vsa_shape_t)
        _lib.vsa_strerror.restype = C.c_char_p
        _lib.vsa_strerror.argtypes = [C.c_int]
        _lib.vsa_workspace_bytes.restype = sz
        _lib.vsa_workspace_bytes.argtypes = [shp, i32, i32, C.c_int]
        _lib.vsa_build_page_summaries.argtypes = [shp, vp, vp, vp, vp, vp, vp]
        _lib.vsa_route_pages.argtypes = [shp, vp, vp, vp, vp, i32, vp, vp, vp, sz, vp]
        _lib.vsa_decode_step_group_shared.argtypes = [shp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, vp, vp, vp, vp,
                                                      vp, vp, sz, vp]
        _lib.vsa_cp_token_candidates.argtypes = [shp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]
        _lib.vsa_cp_partial_readout.argtypes = [shp, vp, vp, vp, vp, vp, i32, f32, vp, vp, vp]
        _lib.vsa_build_super_summaries.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp]
        _lib.vsa_route_pages_two_level.argtypes = [shp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, sz, vp]
        _lib.vsa_decode_step_two_level.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, f32, f32,
                                                   vp, vp, vp, vp, vp, vp, sz, vp]
        _lib.vsa_route_pages_static.argtypes = [shp, vp, vp, vp, vp, i32, vp, vp, vp]
        _lib.vsa_route_pages_static.restype = C.c_int
        _lib.vsa_build_page_summaries_fp8.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp]
        _lib.vsa_sparse_decode_fp8.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, vp, vp, vp, vp, vp]
        _lib.vsa_dense_decode_fallback_fp8.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, vp, f32, vp, vp, vp, sz, vp]
        _lib.vsa_decode_step_fp8.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, vp, vp, vp, vp, vp,
                                             vp, sz, vp]
        _lib.vsa_sparse_decode.argtypes = [shp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, vp, vp, vp, vp, vp, sz, vp]
        _lib.vsa_dense_decode_fallback.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, f32, vp, vp, vp, sz, vp]
        _lib.vsa_decode_step.argtypes = [shp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, vp, vp, vp, vp, vp, vp, sz, vp]
        _lib.vsa_decode_step_timed.argtypes = [shp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, vp, vp, vp, vp, vp, vp, sz,
                                               vp, C.POINTER(C.c_void_p)]
        _lib.vsa_decode_step_host.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32,
                                              vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        _lib.vsa_sparse_decode_entropic.argtypes = [shp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, i32, vp, vp, vp,
                                                    vp, vp, vp]
        _lib.vsa_sparse_decode_frank_wolfe.argtypes = [shp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, i32, vp, vp,
                                                       vp, vp, vp, vp]
        _lib.vsa_decode_step_frank_wolfe.argtypes = [shp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, i32, vp, vp, vp,
                                                     vp, vp, vp, vp, sz, vp]
        _lib.vsa_sparse_decode_frank_wolfe.restype = C.c_int
        _lib.vsa_decode_step_frank_wolfe.restype = C.c_int
        _lib.vsa_decode_step_entropic.argtypes = [shp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, i32, vp, vp, vp,
                                                  vp, vp, vp, vp, sz, vp]
        _lib.vsa_build_page_radii.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp]
        _lib.vsa_decode_step_certified.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, vp, vp, vp, vp,
                                                   vp, vp, vp, sz, vp]
        _lib.vsa_append_kv.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        _lib.vsa_append_kv.restype = C.c_int
        _lib.vsa_decode_step_certified_expand.argtypes = [shp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, f32, f32, vp,
                                                          vp, vp, vp, vp, vp, vp, sz, vp]
        _lib.vsa_decode_step_certified_expand.restype = C.c_int
        _lib.vsa_build_page_radii.restype = C.c_int
        _lib.vsa_decode_step_certified.restype = C.c_int
        for name in ("vsa_build_page_summaries", "vsa_route_pages", "vsa_sparse_decode",
                     "vsa_dense_decode_fallback", "vsa_decode_step", "vsa_decode_step_timed",
                     "vsa_decode_step_host", "vsa_sparse_decode_entropic", "vsa_decode_step_entropic"):
            getattr(_lib, name).restype = C.c_int
    return _lib


def make_shape(batch: int, n_q_heads: int, n_kv_heads: int, max_pages_per_seq: int, num_pool_pages: int,
               head_dim: int = 128, page_size: int = 16, kv_page_stride: int = 0, kv_head_stride: int = 0,
               kv_token_stride: int = 0) -> vsa_shape_t:
    return vsa_shape_t(batch, n_q_heads, n_kv_heads, head_dim, page_size, max_pages_per_seq, num_pool_pages,
                       kv_page_stride, kv_head_stride, kv_token_stride)


def shape_of(q: torch.Tensor, k_cache: torch.Tensor, block_table: torch.Tensor) -> vsa_shape_t:
    """Shape struct for q [B, Hq, d], k_cache [pool, Hkv, page, d] (any strides), block_table [B, max_pages]."""
    assert k_cache.stride(3) == 1, "head dimension must be contiguous"
    return make_shape(q.shape[0], q.shape[1], k_cache.shape[1], block_table.shape[1], k_cache.shape[0],
                      head_dim=q.shape[2], page_size=k_cache.shape[2], kv_page_stride=k_cache.stride(0),
                      kv_head_stride=k_cache.stride(1), kv_token_stride=k_cache.stride(2))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(rc: int, where: str) -> None:
    if rc != 0:
        raise VsaError(rc, where)


def vsa_strerror(code: int) -> str:
    return lib().vsa_strerror(code).decode()


def vsa_workspace_bytes(shape: vsa_shape_t, P: int, K_c: int, which_call: int) -> int:
    return int(lib().vsa_workspace_bytes(C.byref(shape), P, K_c, which_call))


def vsa_build_page_summaries(shape, k_cache, block_table, seq_lens, first_page, summaries, stream=None) -> None:
    _check(lib().vsa_build_page_summaries(C.byref(shape), _ptr(k_cache), _ptr(block_table), _ptr(seq_lens),
                                          _ptr(first_page), _ptr(summaries), _stream(stream)),
           "vsa_build_page_summaries")


def vsa_route_pages(shape, q, summaries, block_table, seq_lens, P, routed_pages, routed_scores, ws,
                    stream=None) -> None:
    _check(lib().vsa_route_pages(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(block_table), _ptr(seq_lens), P,
                                 _ptr(routed_pages), _ptr(routed_scores), _ptr(ws),
                                 0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_route_pages")


def vsa_decode_step_group_shared(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                                 gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws,
                                 stream=None) -> None:
    _check(lib().vsa_decode_step_group_shared(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(k_cache), _ptr(v_cache),
                                              _ptr(block_table), _ptr(seq_lens), P, K_c, epsilon, gap_threshold,
                                              _ptr(out), _ptr(diag), _ptr(routed_pages), _ptr(fallback_list),
                                              _ptr(fallback_count), _ptr(ws),
                                              0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_decode_step_group_shared")


def n_super_pages(shape: vsa_shape_t) -> int:
    return (shape.max_pages_per_seq + VSA_SUPER_PAGES - 1) // VSA_SUPER_PAGES


def vsa_build_super_summaries(shape, summaries, block_table, seq_lens, first_super, super_summaries,
                              super_rep=None, stream=None) -> None:
    _check(lib().vsa_build_super_summaries(C.byref(shape), _ptr(summaries), _ptr(block_table), _ptr(seq_lens),
                                           _ptr(first_super), _ptr(super_summaries), _ptr(super_rep),
                                           _stream(stream)),
           "vsa_build_super_summaries")


def vsa_route_pages_two_level(shape, q, summaries, super_summaries, block_table, seq_lens, P_super, P,
                              routed_pages, routed_scores, super_routed, ws, stream=None) -> None:
    _check(lib().vsa_route_pages_two_level(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(super_summaries),
                                           _ptr(block_table), _ptr(seq_lens), P_super, P, _ptr(routed_pages),
                                           _ptr(routed_scores), _ptr(super_routed), _ptr(ws),
                                           0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_route_pages_two_level")


def vsa_decode_step_two_level(shape, q, summaries, super_summaries, k_cache, v_cache, block_table, seq_lens,
                              P_super, P, K_c, epsilon, gap_threshold, out, diag, routed_pages, fallback_list,
                              fallback_count, ws, stream=None) -> None:
    _check(lib().vsa_decode_step_two_level(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(super_summaries),
                                           _ptr(k_cache), _ptr(v_cache), _ptr(block_table), _ptr(seq_lens),
                                           P_super, P, K_c, epsilon, gap_threshold, _ptr(out), _ptr(diag),
                                           _ptr(routed_pages), _ptr(fallback_list), _ptr(fallback_count), _ptr(ws),
                                           0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_decode_step_two_level")


VSA_STATIC_ROUTE_SCORES = 1 << 20


def vsa_cp_token_candidates(shape, q, k_cache, block_table, seq_lens, routed_pages, P, K_out, cand_pos, cand_score,
                            stream=None) -> None:
    _check(lib().vsa_cp_token_candidates(C.byref(shape), _ptr(q), _ptr(k_cache), _ptr(block_table), _ptr(seq_lens),
                                         _ptr(routed_pages), P, K_out, _ptr(cand_pos), _ptr(cand_score),
                                         _stream(stream)),
           "vsa_cp_token_candidates")


def vsa_cp_partial_readout(shape, v_cache, block_table, seq_lens, cand_pos, cand_score, K_c, epsilon, out_partial,
                           lse_partial, stream=None) -> None:
    _check(lib().vsa_cp_partial_readout(C.byref(shape), _ptr(v_cache), _ptr(block_table), _ptr(seq_lens),
                                        _ptr(cand_pos), _ptr(cand_score), K_c, epsilon, _ptr(out_partial),
                                        _ptr(lse_partial), _stream(stream)),
           "vsa_cp_partial_readout")


def vsa_route_pages_static(shape, q, summaries, block_table, seq_lens, P, routed_pages, routed_scores,
                           stream=None) -> None:
    """vsa_route_pages for callers that have no device memory to lend (a backend inside an engine whose
    pool owns all of HBM, a loop where allocation is banned): the score scratch is a fixed 4 MiB array
    inside the library, so no workspace is passed and nothing is allocated.  Shapes with
    batch * n_q_heads * max_pages_per_seq > VSA_STATIC_ROUTE_SCORES raise VsaError (-6).  Calls share the
    array: do not let two of them overlap on the GPU.  Make the first call on a device outside stream
    capture (it looks up the array's address)."""
    _check(lib().vsa_route_pages_static(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(block_table),
                                        _ptr(seq_lens), P, _ptr(routed_pages), _ptr(routed_scores),
                                        _stream(stream)),
           "vsa_route_pages_static")


def vsa_sparse_decode(shape, q, k_cache, v_cache, block_table, seq_lens, routed_pages, P, K_c, epsilon,
                      gap_threshold, out, diag, fallback_list, fallback_count, ws=None, stream=None) -> None:
    _check(lib().vsa_sparse_decode(C.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                   _ptr(seq_lens), _ptr(routed_pages), P, K_c, epsilon, gap_threshold, _ptr(out),
                                   _ptr(diag), _ptr(fallback_list), _ptr(fallback_count), _ptr(ws),
                                   0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_sparse_decode")


def vsa_dense_decode_fallback(shape, q, k_cache, v_cache, block_table, seq_lens, fallback_list, fallback_count,
                              epsilon, out, diag, ws, stream=None) -> None:
    _check(lib().vsa_dense_decode_fallback(C.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                           _ptr(block_table), _ptr(seq_lens), _ptr(fallback_list),
                                           _ptr(fallback_count), epsilon, _ptr(out), _ptr(diag), _ptr(ws),
                                           0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_dense_decode_fallback")


def vsa_decode_step(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon, gap_threshold,
                    out, diag, routed_pages, fallback_list, fallback_count, ws, stream=None) -> None:
    _check(lib().vsa_decode_step(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(k_cache), _ptr(v_cache),
                                 _ptr(block_table), _ptr(seq_lens), P, K_c, epsilon, gap_threshold, _ptr(out),
                                 _ptr(diag), _ptr(routed_pages), _ptr(fallback_list), _ptr(fallback_count),
                                 _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_decode_step")


# ---- fp8 (e4m3) KV cache: uint8 caches with fp32 scales [pool pages][n_kv_heads]; the shape's strides are bytes ----

def vsa_build_page_summaries_fp8(shape, k_cache, k_scale, block_table, seq_lens, first_page, summaries,
                                 stream=None) -> None:
    _check(lib().vsa_build_page_summaries_fp8(C.byref(shape), _ptr(k_cache), _ptr(k_scale), _ptr(block_table),
                                              _ptr(seq_lens), _ptr(first_page), _ptr(summaries), _stream(stream)),
           "vsa_build_page_summaries_fp8")


def vsa_sparse_decode_fp8(shape, q, k_cache, v_cache, k_scale, v_scale, block_table, seq_lens, routed_pages, P, K_c,
                          epsilon, gap_threshold, out, diag, fallback_list, fallback_count, stream=None) -> None:
    _check(lib().vsa_sparse_decode_fp8(C.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(k_scale),
                                       _ptr(v_scale), _ptr(block_table), _ptr(seq_lens), _ptr(routed_pages), P, K_c,
                                       epsilon, gap_threshold, _ptr(out), _ptr(diag), _ptr(fallback_list),
                                       _ptr(fallback_count), _stream(stream)),
           "vsa_sparse_decode_fp8")


def vsa_dense_decode_fallback_fp8(shape, q, k_cache, v_cache, k_scale, v_scale, block_table, seq_lens, fallback_list,
                                  fallback_count, epsilon, out, diag, ws, stream=None) -> None:
    _check(lib().vsa_dense_decode_fallback_fp8(C.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(k_scale),
                                               _ptr(v_scale), _ptr(block_table), _ptr(seq_lens), _ptr(fallback_list),
                                               _ptr(fallback_count), epsilon, _ptr(out), _ptr(diag), _ptr(ws),
                                               0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_dense_decode_fallback_fp8")


def vsa_decode_step_fp8(shape, q, summaries, k_cache, v_cache, k_scale, v_scale, block_table, seq_lens, P, K_c, epsilon,
                        gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, stream=None) -> None:
    _check(lib().vsa_decode_step_fp8(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(k_cache), _ptr(v_cache),
                                     _ptr(k_scale), _ptr(v_scale), _ptr(block_table), _ptr(seq_lens), P, K_c, epsilon,
                                     gap_threshold, _ptr(out), _ptr(diag), _ptr(routed_pages), _ptr(fallback_list),
                                     _ptr(fallback_count), _ptr(ws),
                                     0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_decode_step_fp8")


def vsa_sparse_decode_entropic(shape, q, k_cache, v_cache, block_table, seq_lens, routed_pages, P, K_c, epsilon,
                               gap_threshold, solver_iters, out, diag, solve, fallback_list, fallback_count,
                               stream=None) -> None:
    _check(lib().vsa_sparse_decode_entropic(C.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                            _ptr(block_table), _ptr(seq_lens), _ptr(routed_pages), P, K_c, epsilon,
                                            gap_threshold, solver_iters, _ptr(out), _ptr(diag), _ptr(solve),
                                            _ptr(fallback_list), _ptr(fallback_count), _stream(stream)),
           "vsa_sparse_decode_entropic")


def vsa_sparse_decode_frank_wolfe(shape, q, k_cache, v_cache, block_table, seq_lens, routed_pages, P, K_c, epsilon,
                                  gap_threshold, solver_iters, out, diag, solve, fallback_list, fallback_count,
                                  stream=None) -> None:
    _check(lib().vsa_sparse_decode_frank_wolfe(C.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                               _ptr(block_table), _ptr(seq_lens), _ptr(routed_pages), P, K_c,
                                               epsilon, gap_threshold, solver_iters, _ptr(out), _ptr(diag),
                                               _ptr(solve), _ptr(fallback_list), _ptr(fallback_count),
                                               _stream(stream)),
           "vsa_sparse_decode_frank_wolfe")


def vsa_decode_step_frank_wolfe(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                                gap_threshold, solver_iters, out, diag, solve, routed_pages, fallback_list,
                                fallback_count, ws, stream=None) -> None:
    _check(lib().vsa_decode_step_frank_wolfe(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(k_cache), _ptr(v_cache),
                                             _ptr(block_table), _ptr(seq_lens), P, K_c, epsilon, gap_threshold,
                                             solver_iters, _ptr(out), _ptr(diag), _ptr(solve), _ptr(routed_pages),
                                             _ptr(fallback_list), _ptr(fallback_count), _ptr(ws),
                                             0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_decode_step_frank_wolfe")


def vsa_decode_step_entropic(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                             gap_threshold, solver_iters, out, diag, solve, routed_pages, fallback_list,
                             fallback_count, ws, stream=None) -> None:
    _check(lib().vsa_decode_step_entropic(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(k_cache), _ptr(v_cache),
                                          _ptr(block_table), _ptr(seq_lens), P, K_c, epsilon, gap_threshold,
                                          solver_iters, _ptr(out), _ptr(diag), _ptr(solve), _ptr(routed_pages),
                                          _ptr(fallback_list), _ptr(fallback_count), _ptr(ws),
                                          0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_decode_step_entropic")


def vsa_build_page_radii(shape, k_cache, summaries, block_table, seq_lens, first_page, radii, stream=None) -> None:
    _check(lib().vsa_build_page_radii(C.byref(shape), _ptr(k_cache), _ptr(summaries), _ptr(block_table),
                                      _ptr(seq_lens), _ptr(first_page), _ptr(radii), _stream(stream)),
           "vsa_build_page_radii")


def vsa_append_kv(shape, k_new, v_new, k_cache, v_cache, block_table, seq_lens, summaries, radii=None,
                  stream=None) -> None:
    _check(lib().vsa_append_kv(C.byref(shape), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache),
                               _ptr(block_table), _ptr(seq_lens), _ptr(summaries), _ptr(radii), _stream(stream)),
           "vsa_append_kv")


def vsa_decode_step_certified(shape, q, summaries, radii, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                              gap_threshold, out, diag, cert, routed_pages, fallback_list, fallback_count, ws,
                              stream=None) -> None:
    _check(lib().vsa_decode_step_certified(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(radii), _ptr(k_cache),
                                           _ptr(v_cache), _ptr(block_table), _ptr(seq_lens), P, K_c, epsilon,
                                           gap_threshold, _ptr(out), _ptr(diag), _ptr(cert), _ptr(routed_pages),
                                           _ptr(fallback_list), _ptr(fallback_count), _ptr(ws),
                                           0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_decode_step_certified")


def vsa_decode_step_certified_expand(shape, q, summaries, radii, k_cache, v_cache, block_table, seq_lens, P, P_expand,
                                     K_c, epsilon, gap_threshold, out, diag, cert, routed_pages, fallback_list,
                                     fallback_count, ws, stream=None) -> None:
    _check(lib().vsa_decode_step_certified_expand(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(radii),
                                                  _ptr(k_cache), _ptr(v_cache), _ptr(block_table), _ptr(seq_lens),
                                                  P, P_expand, K_c, epsilon, gap_threshold, _ptr(out), _ptr(diag),
                                                  _ptr(cert), _ptr(routed_pages), _ptr(fallback_list),
                                                  _ptr(fallback_count), _ptr(ws),
                                                  0 if ws is None else ws.numel() * ws.element_size(),
                                                  _stream(stream)),
           "vsa_decode_step_certified_expand")


def vsa_decode_step_timed(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                          gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, events,
                          stream=None) -> None:
    """`events`: 5 torch.cuda.Event(enable_timing=True) that have been recorded once (so that their
    CUDA handles exist); they are re-recorded between the kernels of the step."""
    handles = (C.c_void_p * 5)(*[e.cuda_event for e in events])
    _check(lib().vsa_decode_step_timed(C.byref(shape), _ptr(q), _ptr(summaries), _ptr(k_cache), _ptr(v_cache),
                                       _ptr(block_table), _ptr(seq_lens), P, K_c, epsilon, gap_threshold,
                                       _ptr(out), _ptr(diag), _ptr(routed_pages), _ptr(fallback_list),
                                       _ptr(fallback_count), _ptr(ws),
                                       0 if ws is None else ws.numel() * ws.element_size(), _stream(stream),
                                       handles),
           "vsa_decode_step_timed")


def vsa_decode_step_host(shape, q_host, q_dev, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c,
                         epsilon, gap_threshold, out_host, out_dev, diag_host, diag_dev, routed_pages,
                         fallback_list, fallback_count, ws, stream=None) -> None:
    _check(lib().vsa_decode_step_host(C.byref(shape), _ptr(q_host), _ptr(q_dev), _ptr(summaries), _ptr(k_cache),
                                      _ptr(v_cache), _ptr(block_table), _ptr(seq_lens), P, K_c, epsilon,
                                      gap_threshold, _ptr(out_host), _ptr(out_dev), _ptr(diag_host),
                                      _ptr(diag_dev), _ptr(routed_pages), _ptr(fallback_list),
                                      _ptr(fallback_count), _ptr(ws),
                                      0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "vsa_decode_step_host")


# ---- small conveniences for callers (allocation and unpacking only) --------------------------------

def alloc_diag(units: int, device) -> torch.Tensor:
    """Device buffer for `units` vsa_diag_t records, viewed as int32 [units, 8]."""
    return torch.zeros((units, DIAG_BYTES // 4), dtype=torch.int32, device=device)


CERT_FIELDS = ("delta_cert", "ub_unrouted", "leak_bound_cert", "certified")


def alloc_cert(units: int, device) -> torch.Tensor:
    """Device buffer for `units` vsa_cert_t records, viewed as int32 [units, 4] (see cert_to_dict)."""
    return torch.zeros((units, 4), dtype=torch.int32, device=device)


def cert_to_dict(cert: torch.Tensor) -> dict:
    c = cert.detach().cpu()
    out = {name: c[:, i].contiguous().view(torch.float32).clone() for i, name in enumerate(CERT_FIELDS[:3])}
    out["certified"] = c[:, 3].clone()
    return out


SOLVE_FIELDS = ("fw_gap", "objective", "residual2", "step")
VSA_SOLVER_MAX_CANDIDATES = 256


def alloc_solve(units: int, device) -> torch.Tensor:
    """Device buffer for `units` vsa_solve_t records: float32 [units, 4], columns = SOLVE_FIELDS."""
    return torch.zeros((units, len(SOLVE_FIELDS)), dtype=torch.float32, device=device)


def diag_to_dict(diag: torch.Tensor) -> dict:
    """Unpack a [units, 8] int32 diag buffer into named host tensors."""
    d = diag.detach().cpu()
    out = {}
    for i, name in enumerate(DIAG_FIELDS):
        col = d[:, i].contiguous()
        out[name] = col.view(torch.float32).clone() if i < 5 else col.clone()
    return out


def alloc_workspace(shape: vsa_shape_t, P: int, K_c: int, which_call: int, device) -> torch.Tensor:
    n = vsa_workspace_bytes(shape, P, K_c, which_call)
    return torch.empty(max(n, 16), dtype=torch.uint8, device=device)
