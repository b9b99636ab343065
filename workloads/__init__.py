"""Seeded synthetic inputs for the sparse paged decode-attention step.

This package only draws random tensors and lays them out as a paged KV cache.
It contains none of the method's arithmetic (no summaries, no scores, no
softmax): the CPU oracle and the CUDA library each consume the bytes produced
here and implement everything else on their own.
"""
from .generator import (  # noqa: F401
    CONFIGS,
    Workload,
    WorkloadSpec,
    config_spec,
    make_workload,
    quantize_kv_fp8,
    seed_for,
)
