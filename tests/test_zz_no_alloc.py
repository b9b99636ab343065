"""vsa_route_pages_static: page routing for callers that cannot hand the library any device memory
(an attention backend inside a serving engine whose pool already owns all of HBM, or a decode loop
in which allocation calls are forbidden).  Its score scratch is a fixed array inside the library, so
the call takes no workspace and allocates nothing.

The test calls it through the C ABI twice in a row - first on a long sequence batch, then on a
shorter one, so that the second call runs on top of whatever the first left in the shared array -
and requires exactly the routed pages and scores that vsa_route_pages produces with a caller-owned
workspace (both are bit-exact by contract, so the tolerance is zero).  It also checks that a shape
beyond the array's capacity is refused on the host.  This file sorts last on purpose: a run that
stops at the first failure has then already exercised every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2602_13804_b200 import binding as B
from workloads import WorkloadSpec, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _route_both_ways(spec, seed):
    w = make_workload(spec, seed=seed).to(DEV)
    shape = B.shape_of(w.q, w.k_cache, w.block_table)
    summ = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, 128), dtype=torch.bfloat16, device=DEV)
    B.vsa_build_page_summaries(shape, w.k_cache, w.block_table, w.seq_lens, None, summ)
    P = spec.P
    want_pages = torch.full((shape.batch, shape.n_q_heads, P), -9, dtype=torch.int32, device=DEV)
    want_scores = torch.zeros((shape.batch, shape.n_q_heads, P), dtype=torch.float32, device=DEV)
    ws = B.alloc_workspace(shape, P, 0, B.VSA_WS_ROUTE, DEV)
    B.vsa_route_pages(shape, w.q, summ, w.block_table, w.seq_lens, P, want_pages, want_scores, ws)
    got_pages = torch.full_like(want_pages, -9)
    got_scores = torch.zeros_like(want_scores)
    B.vsa_route_pages_static(shape, w.q, summ, w.block_table, w.seq_lens, P, got_pages, got_scores)
    torch.cuda.synchronize()
    return want_pages.cpu().numpy(), want_scores.cpu().numpy(), got_pages.cpu().numpy(), got_scores.cpu().numpy()


def test_static_scratch_routing_matches_workspace_routing_on_two_calls_in_a_row():
    long_spec = WorkloadSpec(name="noalloc_long", config=7, batch=3, n_q_heads=8, n_kv_heads=2, P=12, K_c=64,
                             seq_lens=(16 * 700 + 3, 16 * 333, 5000), needles=4)
    short_spec = WorkloadSpec(name="noalloc_short", config=7, batch=3, n_q_heads=8, n_kv_heads=2, P=12, K_c=64,
                              seq_lens=(900, 40, 2049), needles=2)
    for spec, seed in ((long_spec, 71), (short_spec, 72)):
        want_pages, want_scores, got_pages, got_scores = _route_both_ways(spec, seed)
        assert np.array_equal(got_pages, want_pages)
        assert np.array_equal(got_scores, want_scores)
        assert (want_pages >= -1).all() and (want_pages[:, :, 0] >= 0).all()


def test_static_scratch_routing_refuses_shapes_beyond_its_capacity():
    lib = B.lib()
    fake = 0x10000   # never dereferenced: the size check fails on the host first
    too_big = B.make_shape(64, 64, 8, 8192, 1 << 20)          # 64 * 64 * 8192 scores > 2^20
    rc = lib.vsa_route_pages_static(C.byref(too_big), fake, fake, fake, fake, 32, fake, None, None)
    assert rc == -6 and "scratch" in B.vsa_strerror(rc)
    fits = B.make_shape(8, 32, 8, 4096, 1 << 16)               # exactly 2^20 scores
    assert lib.vsa_route_pages_static(C.byref(fits), None, fake, fake, fake, 32, fake, None, None) == -1
