"""Shared helpers for the tests: conversions between torch tensors and the oracle's numpy views."""
import numpy as np
import torch

import oracle
from workloads import Workload


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 bit patterns on the host."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def geometry(w: Workload) -> oracle.Geometry:
    s = w.spec
    return oracle.Geometry(batch=s.batch, n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads,
                           max_pages_per_seq=w.max_pages_per_seq, num_pool_pages=w.pool_pages,
                           head_dim=s.head_dim, page_size=s.page_size)


def host_arrays(w: Workload):
    """(q, K, V, block_table, seq_lens) as the oracle wants them."""
    return (bits(w.q), bits(w.k_cache), bits(w.v_cache),
            w.block_table.cpu().numpy().astype(np.int32), w.seq_lens.cpu().numpy().astype(np.int32))


def gathered_kv(w: Workload, b: int, g: int):
    """fp64 [T, d] keys and values of one (sequence, kv head), in token order."""
    T = int(w.seq_lens[b])
    bs = w.spec.page_size
    n = (T + bs - 1) // bs
    pages = w.block_table[b, :n].long().cpu()
    k = w.k_cache.cpu()[pages, g].reshape(n * bs, -1)[:T].double()
    v = w.v_cache.cpu()[pages, g].reshape(n * bs, -1)[:T].double()
    return k, v
