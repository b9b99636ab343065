"""Sparse paged decode attention for NVIDIA B200: C-ABI CUDA library (libvsa.so) + ctypes binding.

`binding` mirrors include/vsa.h one to one; `engine.SparsePagedDecoder` only owns the device
buffers a caller needs around those calls.  Nothing here computes any step of the path in Python.
"""
from . import binding  # noqa: F401
from .binding import (  # noqa: F401
    VsaError,
    vsa_build_page_summaries,
    vsa_decode_step,
    vsa_decode_step_host,
    vsa_dense_decode_fallback,
    vsa_route_pages,
    vsa_sparse_decode,
    vsa_strerror,
    vsa_workspace_bytes,
)
from .engine import SparsePagedDecoder  # noqa: F401
