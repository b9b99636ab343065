"""Host-side accounting of bench.py (no GPU): the algorithmic bytes per launch follow the union-over-the-
group definition, and the roofline fractions are bytes / time / peak."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from workloads import WorkloadSpec  # noqa: E402


def _spec():
    return WorkloadSpec(name="acc", config=9, batch=2, n_q_heads=4, n_kv_heads=2, P=3, K_c=5, seq_lens=(100, 40))


def test_union_bytes_count_each_page_and_row_once_per_group():
    spec = _spec()
    sl = np.array([100, 40])                       # 7 and 3 pages
    # routed pages [B, Hq, P]: heads 0,1 form group 0, heads 2,3 group 1
    rp = np.array([[[0, 1, 2], [1, 2, 3], [5, 6, -1], [5, 6, -1]],
                   [[0, 1, -1], [0, 1, -1], [2, -1, -1], [1, 2, -1]]])
    # candidate positions [B, Hq, K_c]
    cp = np.array([[[0, 1, 2, 3, 4], [3, 4, 5, 6, 7], [80, 81, -1, -1, -1], [80, 82, -1, -1, -1]],
                   [[0, 1, 2, 3, 4], [0, 1, 2, 3, 4], [33, -1, -1, -1, -1], [17, 33, -1, -1, -1]]])
    fb = np.array([[0, 1, 0, 0], [0, 0, 0, 0]])
    a = bench.algorithmic_bytes(spec, sl, rp, cp, fb)
    union_pages = 4 + 2 + 2 + 2                     # {0,1,2,3}, {5,6}, {0,1}, {1,2}
    union_rows = 8 + 3 + 5 + 2                      # {0..7}, {80,81,82}, {0..4}, {17,33}
    assert a["sparse_union_pages"] == union_pages and a["sparse_union_rows"] == union_rows
    units = 8
    assert a["sparse_decode"] == union_pages * 16 * 256 + union_rows * 256 + units * (256 + 512)
    # scan: one 256-byte summary row per (page, KV head) + a block-table entry per page + q
    assert a["route_scan"] == (7 + 3) * (2 * 256 + 4) + units * 256
    # dense: K and V rows of every (sequence, KV head) with a flagged head
    assert a["dense_fallback"] == 100 * 2 * 256
    # the paper's per-query-head model books every head's pages and rows
    per_head = ((3 * 16 + 5) * 256) * 4 + ((3 * 16 + 5) * 256) * 4 + units * 768
    assert a["sparse_decode_per_head_model"] == per_head


def test_fractions_are_bytes_over_time_over_peak():
    alg = {"route_scan": 10_000_000, "sparse_decode": 5_000_000, "sparse_decode_per_head_model": 20_000_000,
           "dense_fallback": 0}
    pk = {"route_scan": 10.0, "event_pair_overhead": 2.0, "sparse_decode": 5.0, "dense_fallback": 1.0}
    k = bench.kernel_fracs(alg, pk, 12.5, 5000.0)
    assert abs(k["route_scan"]["achieved_GBps"] - 1000.0) < 1e-9 and abs(k["route_scan"]["frac"] - 0.2) < 1e-12
    assert abs(k["sparse_decode"]["frac"] - 0.2) < 1e-12 and abs(k["sparse_decode"]["frac_per_head_model"] - 0.8) < 1e-12
    assert abs(k["step"]["achieved_GBps"] - 15_000_000 / 12.5e-6 / 1e9) < 1e-9
    assert abs(k["sparse_decode"]["frac_of_8TBps"] - 1000.0 / 8000.0) < 1e-12
