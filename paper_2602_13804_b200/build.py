"""Builds libvsa.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Usage: python -m paper_2602_13804_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libvsa.so")
SOURCES = ["api.cu", "summaries.cu", "route.cu", "two_level.cu", "sparse.cu", "sparse_plain.cu", "sparse_plain_d64.cu", "sparse_plain_d256.cu", "sparse_plain_fp8.cu", "sparse_solve.cu", "sparse_cert.cu", "sparse_two_level.cu", "sparse_shared_g12.cu", "sparse_shared_g4.cu", "sparse_shared_g8.cu",
           "dense.cu", "context_parallel.cu"]
HEADERS = ["vsa_device.cuh", "vsa_select.cuh", "sparse_kernel.cuh", "sparse_shared.cuh", "vsa_team.cuh", "vsa_launch.h", os.path.join("..", "..", "include", "vsa.h")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "--threads", "0",
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", tmp,
           *[os.path.join(CSRC, s) for s in SOURCES]]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
