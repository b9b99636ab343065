#!/usr/bin/env python
"""Benchmark of the sparse paged decode-attention step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A "step" is one decode token for every sequence of the batch through all layers of the
workload: per layer vsa_decode_step (page routing -> fused sparse pass -> dense fallback) on
that layer's own KV cache.  Prints ONE JSON line (rank 0).  Workloads:
    cfg1            batch 8, T = 32768, 32 layers, P = 32, K_c = 256  (default; the metric's config)
    cfg0 | cfg3 | cfg4
    cfg2:B:T        a point of the context sweep, e.g. cfg2:1:131072
With --gpus N > 1 and no torchrun environment the script starts its N ranks itself
(python -m torch.distributed.run ... bench.py, one process per GPU, no data-path collective).
Extra flags: --layers L (override), --dense-baseline (time the split-K dense kernel on the same
caches instead of the sparse path), --no-graph (plain stream launches for `value`), --no-sweep
(skip the context sweep / fallback / scan points that the default run adds to its line),
--grid (the (P, K_c) ablation grid of the paper's Table 3 as one JSON line),
--leak-curve (leakage against the gap statistic, CPU oracle only, one JSON line).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attn_us_per_token_per_layer"
UNIT = "us/token/layer"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0      # the denominator the metric names ("vs 8 TB/s")
SUSTAIN_S = 0.6               # length of the event-timed region the clock samples come from


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg1")
    ap.add_argument("--layers", type=int, default=None)
    ap.add_argument("--dense-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--grid", action="store_true",
                    help="time the (P, K_c) grid of the paper's Table 3 at batch 8, T = 65536 and print it")
    ap.add_argument("--leak-curve", action="store_true",
                    help="leakage against the gap statistic on config-0-shaped workloads (CPU oracle only)")
    ap.add_argument("--needle-mode", default=None, choices=["group_sum", "per_qhead_round_robin", "unit_literal"],
                    help="override how the planted keys are aligned with the queries (workloads/generator.py)")
    ap.add_argument("--P", type=int, default=None, help="override the workload's routed pages per unit")
    ap.add_argument("--Kc", type=int, default=None, help="override the workload's candidate count per unit")
    ap.add_argument("--certified", action="store_true",
                    help="time vsa_decode_step_certified (routing certificate computed, certified gap decides the "
                         "fallback) instead of vsa_decode_step")
    ap.add_argument("--expand", type=int, default=None,
                    help="with --certified: retry the refused units with up to this many routed pages before the "
                         "dense pass (vsa_decode_step_certified_expand)")
    ap.add_argument("--two-level", type=int, default=None, metavar="P_SUPER",
                    help="time vsa_decode_step_two_level: only the pages of the P_SUPER best super-pages (16 pages "
                         "each, scored through one representative summary) are scored per unit")
    ap.add_argument("--fp8", action="store_true",
                    help="time vsa_decode_step_fp8 on an e4m3 copy of the workload's caches against vsa_decode_step on the "
                         "bf16 caches that hold the same values, and print that comparison as one JSON line")
    ap.add_argument("--group-shared", action="store_true",
                    help="time vsa_decode_step_group_shared: the heads of a GQA group route as one query (one page "
                         "set and one candidate set per KV head)")
    ap.add_argument("--solver", default="eg", choices=["eg", "fw"],
                    help="with --solver-iters: entropic mirror descent (eg) or Frank-Wolfe with exact line search (fw)")
    ap.add_argument("--solver-iters", type=int, default=None,
                    help="time the step whose candidate weights come from this many entropic mirror-descent "
                         "iterations (vsa_decode_step_entropic) instead of the closed form")
    return ap.parse_args(argv)


def workload_spec(name: str, layers):
    from workloads import config_spec
    if name.startswith("cfg2:"):
        _, b, t = name.split(":")
        spec = config_spec(2, batch=int(b), T=int(t), layers=32, name=f"cfg2_b{b}_t{t}")
    else:
        spec = config_spec(int(name[3:]))
    if spec.layers == 1 and layers is None:
        layers = 32          # every workload is timed over 32 distinct layer caches
    if layers is not None:
        from dataclasses import replace
        spec = replace(spec, layers=int(layers))
    return spec


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0: float, t1: float) -> dict:
        """Summary of the samples taken between the wall-clock times t0 and t1 (the timed region)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        inside = [r for (t, r) in self.rows if t0 <= t <= t1 and len(r) >= 7]
        rows = inside or [r for (_, r) in self.rows if len(r) >= 7]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm = sorted(float(r[0]) for r in rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].lower().startswith("active") for r in rows)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][1]),
                "power_w_max": max(float(r[2]) for r in rows), "reasons": reasons, "samples": len(rows),
                "samples_inside_timed_region": len(inside)}


def max_over_ranks(ms: float, world: int, device) -> float:
    """Time of the slowest rank: every rank decodes its own sequences, the job is done when all are."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def us_per_token_per_layer(ms_per_step: float, world: int, batch_per_rank: int, layers: int) -> float:
    """Whole-job figure: one step decodes world * batch tokens through `layers` layers."""
    return ms_per_step * 1e3 / (world * batch_per_rank * layers)


def spawn_command(args_list, n_gpus: int, port: int):
    """The launch line for N ranks of this script on one node (one process per GPU)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *args_list]


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def host_bits(t):
    import numpy as np
    import torch
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_inputs(w):
    import numpy as np
    import oracle
    s = w.spec
    geo = oracle.Geometry(batch=s.batch, n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads,
                          max_pages_per_seq=w.max_pages_per_seq, num_pool_pages=w.pool_pages)
    q, K, V = host_bits(w.q), host_bits(w.k_cache), host_bits(w.v_cache)
    bt, sl = w.block_table.cpu().numpy().astype(np.int32), w.seq_lens.cpu().numpy().astype(np.int32)
    return geo, q, K, V, bt, sl


def oracle_layer_time(w, reps_budget_s: float = 12.0, dense: bool = False, inputs=None):
    """Times the CPU oracle, as it stands, on one layer of the workload (all sequences).
    Returns (seconds per layer-step, repetitions, threads)."""
    import oracle
    s = w.spec
    geo, q, K, V, bt, sl = inputs or oracle_inputs(w)
    summ = oracle.build_summaries(geo, K, bt, sl)      # cache maintenance, outside the timed step
    reps, t_total = 0, 0.0
    while True:
        t0 = time.perf_counter()
        if dense:
            oracle.dense(geo, q, K, V, bt, sl, w.epsilon)
        else:
            oracle.decode_step(geo, q, K, V, bt, sl, s.P, s.K_c, w.epsilon, w.gap_threshold, summaries=summ)
        t_total += time.perf_counter() - t0
        reps += 1
        if t_total >= reps_budget_s or reps >= 200:
            break
    return t_total / reps, reps, oracle.num_threads()


def algorithmic_bytes(spec, seq_lens, routed_pages=None, cand_pos=None, fallback=None):
    """Bytes one launch of each kernel has to move for this layer ("algorithmic bytes").

    scan:   every owned page's summary row of every KV head + its block-table entry + q.
    sparse: per (sequence, KV head) the UNION over the group's query heads of the routed pages x 4 KB
            (K tiles) and the union of the candidates' value rows x 256 B, + q and out per unit.
            Needs the routed / candidate sets (taken from the oracle's run of the layer); without them
            only the per-query-head model (P * 16 + K_c) * 256 B of the paper's Cor. 3 is returned.
    dense:  K and V rows of every (sequence, KV head) with at least one flagged head, 512 B per token.
    """
    import numpy as np
    sl = np.asarray(seq_lens, dtype=np.int64)
    n_pages = (sl + spec.page_size - 1) // spec.page_size
    B, Hq, Hkv = spec.batch, spec.n_q_heads, spec.n_kv_heads
    G = Hq // Hkv
    units = B * Hq
    row = spec.head_dim * 2
    out = {"route_scan": int(n_pages.sum()) * (Hkv * row + 4) + units * row}
    np_eff = np.minimum(spec.P, n_pages)
    n_cand = np.minimum(spec.K_c, np_eff * spec.page_size)
    out["sparse_decode_per_head_model"] = int(((np_eff * spec.page_size + n_cand) * row).sum()) * Hq + units * (row + 2 * row)
    if routed_pages is not None and cand_pos is not None:
        rp = np.asarray(routed_pages).reshape(B, Hkv, G, -1)
        cp = np.asarray(cand_pos).reshape(B, Hkv, G, -1)
        pages = rows = 0
        for b in range(B):
            for g in range(Hkv):
                p = rp[b, g].reshape(-1)
                c = cp[b, g].reshape(-1)
                pages += np.unique(p[p >= 0]).size
                rows += np.unique(c[c >= 0]).size
        out["sparse_decode"] = pages * spec.page_size * row + rows * row + units * (row + 2 * row)
        out["sparse_union_pages"], out["sparse_union_rows"] = int(pages), int(rows)
    if fallback is not None:
        fb = np.asarray(fallback).reshape(B, Hkv, G).any(axis=2)
        out["dense_fallback"] = int((fb * sl[:, None]).sum()) * 2 * row
    return out


def run_reference(args):
    """The CPU oracle as the reference arm: same workload, metric and unit; each step is a
    bounded sample (one layer of the workload, all sequences)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from workloads import make_workload
    spec = workload_spec(args.workload, args.layers)
    w = make_workload(spec, device="cpu", rep=0)
    import oracle
    s = w.spec
    geo, q, K, V, bt, sl = oracle_inputs(w)
    summ = oracle.build_summaries(geo, K, bt, sl)

    def one():
        oracle.decode_step(geo, q, K, V, bt, sl, s.P, s.K_c, w.epsilon, w.gap_threshold, summaries=summ)

    for _ in range(args.warmup):
        one()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one()
    dt = (time.perf_counter() - t0) / args.steps
    value = dt * 1e6 / s.batch          # one layer per step: us per token per layer
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": spec.name, "batch": s.batch, "n_q_heads": s.n_q_heads, "n_kv_heads": s.n_kv_heads,
                   "P": s.P, "K_c": s.K_c, "step": "one layer of the workload per step (bounded sample)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": "layer 0 of the workload, all sequences, one decode step per timed step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


class Harness:
    """Layer caches, buffers and the captured step of one workload on one GPU."""

    def __init__(self, spec, dev, rank: int = 0, mem_fraction: float = 0.8, args=None):
        import torch
        from paper_2602_13804_b200 import binding as B
        from workloads import make_workload
        self.B, self.torch = B, torch
        self.spec, self.dev, self.args = spec, dev, args
        L = spec.layers
        w0 = make_workload(spec, device=dev, rep=0, sub=rank)
        per_layer = 2 * w0.k_cache.numel() * 2 + w0.pool_pages * spec.n_kv_heads * 256
        free, _ = torch.cuda.mem_get_info(dev)
        self.distinct = max(1, min(L, int(mem_fraction * free // per_layer) + 1))
        self.layers = [w0] + [make_workload(spec, device=dev, rep=i, sub=rank) for i in range(1, self.distinct)]
        self.L = L
        self.shape = B.shape_of(w0.q, w0.k_cache, w0.block_table)
        # A paged KV cache has ONE block table and one length vector per sequence, used by every layer
        # (the layers' K/V pools are separate tensors indexed by the same page numbers): all layers get
        # layer 0's tensors.  The generator gives every layer the same structure, which is checked.
        for w in self.layers:
            assert w.pool_pages == w0.pool_pages and torch.equal(w.block_table, w0.block_table) and \
                torch.equal(w.seq_lens, w0.seq_lens)
            w.block_table, w.seq_lens = w0.block_table, w0.seq_lens
        shape = self.shape
        self.units = shape.batch * shape.n_q_heads
        self.P, self.K_c, self.eps, self.tau = spec.P, spec.K_c, w0.epsilon, w0.gap_threshold

        # cache maintenance (off the decode path): summaries of every layer, timed separately
        self.summaries = []
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for w in self.layers:
            s = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=dev)
            B.vsa_build_page_summaries(shape, w.k_cache, w.block_table, w.seq_lens, None, s)
            self.summaries.append(s)
        ev1.record()
        torch.cuda.synchronize()
        self.summary_ms_per_layer = ev0.elapsed_time(ev1) / len(self.layers)

        P, K_c, units = self.P, self.K_c, self.units
        self.out = torch.empty((shape.batch, shape.n_q_heads, 128), dtype=torch.float32, device=dev)
        self.diag = B.alloc_diag(units, dev)
        self.routed = torch.empty((shape.batch, shape.n_q_heads, P), dtype=torch.int32, device=dev)
        self.flist = torch.empty(units, dtype=torch.int32, device=dev)
        self.fcount = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ws = B.alloc_workspace(shape, P, K_c, B.VSA_WS_STEP, dev)
        self.ws_dense = B.alloc_workspace(shape, P, K_c, B.VSA_WS_DENSE, dev)
        self.ws_plain = self.ws
        self.solve = self.cert = self.radii = None
        self.routed_plain = self.routed
        a = args
        if a is not None and a.solver_iters is not None:
            self.solve = B.alloc_solve(units, dev)
        if a is not None and a.certified:
            self.cert = B.alloc_cert(units, dev)
            self.ws = B.alloc_workspace(shape, a.expand or P, K_c,
                                        B.VSA_WS_STEP_EXPAND if a.expand else B.VSA_WS_STEP_CERTIFIED, dev)
            if a.expand:
                self.routed = torch.empty((shape.batch, shape.n_q_heads, a.expand), dtype=torch.int32, device=dev)
            self.radii = []
            for w, s_ in zip(self.layers, self.summaries):      # cache maintenance, like the summaries
                r = torch.zeros((shape.num_pool_pages, shape.n_kv_heads), dtype=torch.float32, device=dev)
                B.vsa_build_page_radii(shape, w.k_cache, s_, w.block_table, w.seq_lens, None, r)
                self.radii.append(r)
        self.routed_group = torch.empty((shape.batch, shape.n_kv_heads, P), dtype=torch.int32, device=dev)
        self.supers = None
        if a is not None and getattr(a, "two_level", None):
            self.ws = B.alloc_workspace(shape, a.two_level, K_c, B.VSA_WS_STEP_TWO_LEVEL, dev)
            self.supers = []
            for w, s_ in zip(self.layers, self.summaries):      # cache maintenance, like the summaries
                sp = torch.zeros((shape.batch, B.n_super_pages(shape), shape.n_kv_heads, shape.head_dim),
                                 dtype=torch.bfloat16, device=dev)
                B.vsa_build_super_summaries(shape, s_, w.block_table, w.seq_lens, None, sp)
                self.supers.append(sp)
        self.stream = torch.cuda.Stream(device=dev)
        self.graph = None

    # ---- one layer of the step -----------------------------------------------------------------
    def layer_call(self, i, plain=False):
        B, a, shape = self.B, self.args, self.shape
        k = i % self.distinct
        w, s = self.layers[k], self.summaries[k]
        P, K_c, eps, tau = self.P, self.K_c, self.eps, self.tau
        out, diag, routed, flist, fcount, ws = self.out, self.diag, self.routed, self.flist, self.fcount, self.ws
        if a is not None and a.dense_baseline and not plain:
            B.vsa_dense_decode_fallback(shape, w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, None, None,
                                        eps, out, diag, self.ws_dense)
        elif a is not None and getattr(a, "group_shared", False) and not plain:
            B.vsa_decode_step_group_shared(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c, eps,
                                           tau, out, diag, self.routed_group, flist, fcount, self.ws_plain)
        elif self.supers is not None and not plain:
            B.vsa_decode_step_two_level(shape, w.q, s, self.supers[k], w.k_cache, w.v_cache, w.block_table,
                                        w.seq_lens, a.two_level, P, K_c, eps, tau, out, diag, routed, flist, fcount,
                                        ws)
        elif self.cert is not None and a.expand and not plain:
            B.vsa_decode_step_certified_expand(shape, w.q, s, self.radii[k], w.k_cache, w.v_cache, w.block_table,
                                               w.seq_lens, P, a.expand, K_c, eps, tau, out, diag, self.cert, routed,
                                               flist, fcount, ws)
        elif self.cert is not None and not plain:
            B.vsa_decode_step_certified(shape, w.q, s, self.radii[k], w.k_cache, w.v_cache, w.block_table,
                                        w.seq_lens, P, K_c, eps, tau, out, diag, self.cert, routed, flist, fcount, ws)
        elif self.solve is not None and a.solver == "fw" and not plain:
            B.vsa_decode_step_frank_wolfe(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c, eps,
                                          tau, a.solver_iters, out, diag, self.solve, routed, flist, fcount, ws)
        elif self.solve is not None and not plain:
            B.vsa_decode_step_entropic(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c, eps,
                                       tau, a.solver_iters, out, diag, self.solve, routed, flist, fcount, ws)
        else:
            B.vsa_decode_step(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c, eps, tau,
                              out, diag, routed if routed.shape[-1] == P else self.routed_plain, flist, fcount,
                              self.ws_plain)

    def step_plain(self, plain=False):
        for i in range(self.L):
            self.layer_call(i, plain)

    def capture(self, use_graph=True, plain=False):
        """Returns the callable that runs one step (graph replay, or plain launches)."""
        torch = self.torch
        with torch.cuda.stream(self.stream):
            self.step_plain(plain)                # first call: function attributes, lazy module load
            self.stream.synchronize()
            if not use_graph:
                return lambda: self.step_plain(plain)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=self.stream):
                self.step_plain(plain)
        return g.replay

    def time_steps(self, step, n, world=1, barrier=None):
        """ms for n back-to-back steps between two events on the launching stream."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.stream):
            e0.record(self.stream)
            for _ in range(n):
                step()
            e1.record(self.stream)
        if barrier:
            barrier()
        else:
            self.stream.synchronize()
        return max_over_ranks(e0.elapsed_time(e1), world, self.dev)

    def per_kernel(self, step, n_rep):
        """us per launch of each kernel: event intervals around the kernels of the same launch sequence
        (vsa_decode_step_timed).  The interval between two event records holds the kernel plus the cost of
        the records themselves; the second slot of the timed step brackets no kernel (the page selection
        is fused into the sparse kernel) and reads that cost, which is reported, not subtracted."""
        import numpy as np
        torch, B, shape = self.torch, self.B, self.shape
        L = self.L
        with torch.cuda.stream(self.stream):
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(L)]
            for row in evs:
                for e in row:
                    e.record(self.stream)
            acc = np.zeros(4)
            for _ in range(2):
                step()

            def timed_pass():
                for i in range(L):
                    k = i % self.distinct
                    w, s = self.layers[k], self.summaries[k]
                    B.vsa_decode_step_timed(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, self.P,
                                            self.K_c, self.eps, self.tau, self.out, self.diag, self.routed,
                                            self.flist, self.fcount, self.ws, evs[i])
            timed_pass()
            self.stream.synchronize()
            for _ in range(n_rep):
                # hold the GPU for ~3 ms so that the host enqueues the whole step ahead of it:
                # the events then bracket kernels that run back to back, not launch gaps
                torch.cuda._sleep(6_000_000)
                timed_pass()
                self.stream.synchronize()
                for row in evs:
                    acc += np.array([row[j].elapsed_time(row[j + 1]) for j in range(4)])
        return dict(zip(["route_scan", "event_pair_overhead", "sparse_decode", "dense_fallback"],
                        (acc / (n_rep * L) * 1e3).tolist()))    # us per launch

    def fallback_units(self):
        n = int(self.fcount.item())
        return self.flist[:n].cpu().numpy()

    def release(self):
        self.graph = None
        self.layers = self.summaries = self.radii = None
        self.torch.cuda.empty_cache()


def kernel_fracs(alg, per_kernel, step_us, peak):
    """Achieved GB/s and roofline fractions per kernel and for the whole step."""
    def entry(nbytes, us):
        gbs = nbytes / (us * 1e-6) / 1e9 if us > 0 else 0.0
        return {"bytes_per_launch": int(nbytes), "us_per_launch": us, "achieved_GBps": gbs,
                "frac": gbs / peak, "frac_of_8TBps": gbs / NOMINAL_HBM_GBS}
    out = {}
    sparse_key = "sparse_decode" if "sparse_decode" in alg else "sparse_decode_per_head_model"
    names = {"route_scan": "route_scan", "sparse_decode": sparse_key, "dense_fallback": "dense_fallback"}
    total = 0
    for k, a in names.items():
        if a in alg and per_kernel and k in per_kernel:
            out[k] = entry(alg[a], per_kernel[k])
            total += alg[a]
    if sparse_key != "sparse_decode" and "sparse_decode" in out:
        out["sparse_decode"]["bytes_model"] = "per query head (no oracle sets available)"
    if "sparse_decode_per_head_model" in alg and per_kernel and "sparse_decode" in out:
        out["sparse_decode"]["frac_per_head_model"] = \
            alg["sparse_decode_per_head_model"] / (per_kernel["sparse_decode"] * 1e-6) / 1e9 / peak
    out["step"] = entry(total, step_us)
    out["step"]["note"] = "sum of the kernels' algorithmic bytes / graph-replayed us per layer"
    return out


def measure_point(spec, dev, steps, want_kernels=True, use_graph=True, oracle_sets=False):
    """One extra workload (a sweep point): us per layer of the whole step, per-kernel intervals,
    fallback fraction and roofline fractions.  Used by the default run's `sweep` object."""
    import numpy as np
    h = Harness(spec, dev)
    step = h.capture(use_graph)
    with h.torch.cuda.stream(h.stream):
        for _ in range(3):
            step()
    ms = h.time_steps(step, steps)
    us_layer = ms / steps * 1e3 / h.L
    fb = h.fallback_units()
    fallback = np.zeros(h.units, np.int32)
    fallback[fb] = 1
    pk = h.per_kernel(step, 5) if want_kernels else None
    rp = cp = None
    if oracle_sets:
        import oracle
        w0 = h.layers[(h.L - 1) % h.distinct]          # the layer whose fallback list is in the buffers
        geo, q, K, V, bt, sl = oracle_inputs(w0)
        st = oracle.decode_step(geo, q, K, V, bt, sl, spec.P, spec.K_c, w0.epsilon, w0.gap_threshold)
        rp, cp = st.route.pages, st.sparse.cand_pos
    sl = h.layers[0].seq_lens.cpu().numpy()
    alg = algorithmic_bytes(spec, sl, rp, cp, fallback)
    peak, _ = measured_peak()
    point = {"workload": spec.name, "batch": spec.batch, "context": int(sl.max()), "layers": h.L,
             "distinct_layer_caches": h.distinct, "us_per_layer": us_layer,
             "us_per_token_per_layer": us_layer / spec.batch, "fallback_fraction": float(len(fb)) / h.units,
             "per_kernel_us": pk, "kernels": kernel_fracs(alg, pk, us_layer, peak) if pk else None}
    h.release()
    return point


def two_level_point(spec, dev, P_super, steps):
    """The step with two-level routing against the plain step on the same caches, and the fraction of the
    exact routing's pages that the pre-filter keeps (both page lists come from the GPU, last layer)."""
    import numpy as np
    a = parse_args(["--two-level", str(P_super)])
    h = Harness(spec, dev, args=a)
    res = {}
    lists = {}
    for name, plain in (("two_level", False), ("full_scan", True)):
        step = h.capture(True, plain=plain)
        with h.torch.cuda.stream(h.stream):
            for _ in range(3):
                step()
        res[name] = h.time_steps(step, steps) / steps * 1e3 / h.L
        lists[name] = h.routed.cpu().numpy().reshape(h.units, -1)
    hit = tot = 0
    for u in range(h.units):
        e = set(int(x) for x in lists["full_scan"][u] if x >= 0)
        hit += len(e & set(int(x) for x in lists["two_level"][u]))
        tot += len(e)
    h.release()
    return {"workload": spec.name, "P_super": P_super, "us_per_layer": res["two_level"],
            "us_per_layer_full_scan": res["full_scan"], "page_recall_vs_exact_routing": hit / max(tot, 1)}


def fp8_point(spec, dev, steps):
    """The step on an fp8 (e4m3, power-of-two scale per page and KV head) copy of the caches against the bf16
    step on the bf16 caches that hold the same values (same routed pages, candidates and flags by construction)."""
    from workloads import quantize_kv_fp8
    h = Harness(spec, dev, mem_fraction=0.5)
    torch, B, shape = h.torch, h.B, h.shape
    k8s, v8s, kss, vss = [], [], [], []
    for i, w in enumerate(h.layers):
        wq, k8, v8, ke, ve = quantize_kv_fp8(w)
        h.layers[i] = wq                        # the bf16 side runs on the dequantised values
        k8s.append(k8); v8s.append(v8)
        kss.append(torch.exp2(ke.float())); vss.append(torch.exp2(ve.float()))
        B.vsa_build_page_summaries_fp8(shape, k8, kss[-1], wq.block_table, wq.seq_lens, None, h.summaries[i])
    del w, wq
    torch.cuda.synchronize()

    def fp8_step():
        for i in range(h.L):
            k = i % h.distinct
            w = h.layers[k]
            B.vsa_decode_step_fp8(shape, w.q, h.summaries[k], k8s[k], v8s[k], kss[k], vss[k], w.block_table, w.seq_lens,
                                  h.P, h.K_c, h.eps, h.tau, h.out, h.diag, h.routed, h.flist, h.fcount, h.ws_plain)
    res = {}
    with torch.cuda.stream(h.stream):
        fp8_step()
        h.stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=h.stream):
            fp8_step()
        for _ in range(3):
            g.replay()
    res["fp8"] = h.time_steps(g.replay, steps) / steps * 1e3 / h.L
    fb8 = len(h.fallback_units()) / h.units
    st = h.capture(True)
    with torch.cuda.stream(h.stream):
        for _ in range(3):
            st()
    res["bf16"] = h.time_steps(st, steps) / steps * 1e3 / h.L
    fb16 = len(h.fallback_units()) / h.units
    point = {"workload": spec.name, "layers": h.L, "distinct_layer_caches": h.distinct,
             "us_per_layer_fp8": res["fp8"], "us_per_layer_bf16_same_values": res["bf16"],
             "fallback_fraction_fp8": fb8, "fallback_fraction_bf16": fb16}
    h.release()
    return point


def sweep(dev, steps_small=200):
    """The context sweep at batch 1 (flatness), one fallback-regime point and one large scan point."""
    from dataclasses import replace
    from workloads import config_spec
    out = {"batch1": [], "note": "cfg2 at batch 1, P = 32, K_c = 256, 16 distinct layer caches per point "
                                 "(graph replay, device events); flatness = us_per_layer(128k) / us_per_layer(4k)"}
    for T in (4096, 8192, 16384, 32768, 65536, 131072):
        spec = config_spec(2, batch=1, T=T, layers=16, name=f"cfg2_b1_t{T}")
        out["batch1"].append(measure_point(spec, dev, steps_small))
    t = {p["context"]: p["us_per_layer"] for p in out["batch1"]}
    out["flatness"] = t[131072] / t[4096]
    # the small-gap regime: config 3's shape with fewer layer caches so that it fits the run
    spec3 = replace(config_spec(3), layers=4, name="cfg3_fallback_4layers")
    out["fallback_regime"] = measure_point(spec3, dev, 20)
    # the scan where its traffic dominates: batch 16, T = 128k, two layer caches
    spec16 = config_spec(2, batch=16, T=131072, layers=2, name="cfg2_b16_t131072_2layers")
    out["scan_large"] = measure_point(spec16, dev, 40)
    # a multi-query shape: config 1 with ONE KV head for the 32 query heads
    out["mqa"] = measure_point(replace(config_spec(1), n_kv_heads=1, layers=16, name="cfg1_mqa_32q_1kv"), dev, 100)
    # 32-token pages: config 1 with half as many pages routed (the same 512 scored tokens per unit)
    c1 = config_spec(1)
    out["page32"] = measure_point(replace(c1, page_size=32, P=c1.P // 2, layers=16, name="cfg1_page32_halfP"), dev, 100)
    # other head dimensions: config 1's shape at d = 64 and d = 256 (temperature sqrt(d))
    out["head_dims"] = [measure_point(replace(c1, head_dim=d, epsilon=math.sqrt(d), layers=L, name=f"cfg1_d{d}"), dev, 100)
                        for d, L in ((64, 16), (256, 8))]
    # fp8 KV cache against bf16 on the same values: config 1 (no fallback) and config 3's shape (75 % dense)
    out["fp8"] = [fp8_point(replace(c1, layers=8, name="cfg1_8layers"), dev, 100),
                  fp8_point(replace(config_spec(3), layers=2, name="cfg3_fallback_2layers"), dev, 20)]
    # group-shared routing (one selection per KV head) on config 1 and at batch 16
    gs = []
    for spec_g in (replace(config_spec(1), layers=16, name="cfg1_16layers"),
                   config_spec(2, batch=16, T=32768, layers=8, name="cfg2_b16_t32768")):
        a = parse_args(["--group-shared"])
        hg = Harness(spec_g, dev, args=a)
        res = {}
        for name, plain in (("group_shared", False), ("per_head", True)):
            st = hg.capture(True, plain=plain)
            with hg.torch.cuda.stream(hg.stream):
                for _ in range(3):
                    st()
            res[name] = hg.time_steps(st, 50) / 50 * 1e3 / hg.L
        hg.release()
        gs.append({"workload": spec_g.name, "us_per_layer_group_shared": res["group_shared"],
                   "us_per_layer_per_head_routing": res["per_head"]})
    out["group_shared"] = gs
    # the expansion loop where it rescues units: config 1 routed with 8 pages although 32 pages hold a planted
    # key - the certificate refuses every unit; doubling the page budget up to 32 certifies them all
    ex = []
    spec_e = replace(config_spec(1), layers=8, P=8, K_c=128, name="cfg1_8layers_P8_Kc128")
    for flags in (["--certified"], ["--certified", "--expand", "32"]):
        he = Harness(spec_e, dev, args=parse_args(flags))
        st = he.capture(True)
        with he.torch.cuda.stream(he.stream):
            for _ in range(3):
                st()
        us = he.time_steps(st, 20) / 20 * 1e3 / he.L
        ex.append({"flags": " ".join(flags), "us_per_layer": us, "fallback_fraction": len(he.fallback_units()) / he.units})
        he.release()
    out["expansion_rescue"] = {"workload": spec_e.name, "points": ex}
    # two-level routing at batch 16: growth of the step from 4k to 128k against the full scan's
    # (at 4k every super-page is kept, so the call runs the exact step) and at batch 1, T = 128k
    tl = [two_level_point(config_spec(2, batch=16, T=4096, layers=16, name="cfg2_b16_t4096"), dev, 32, 100),
          two_level_point(spec16, dev, 32, 40)]
    out["two_level_b16"] = {"points": tl, "growth_4k_to_128k": tl[1]["us_per_layer"] / tl[0]["us_per_layer"],
                            "growth_4k_to_128k_full_scan": tl[1]["us_per_layer_full_scan"] / tl[0]["us_per_layer_full_scan"]}
    out["two_level_b1"] = [two_level_point(config_spec(2, batch=1, T=T, layers=16, name=f"cfg2_b1_t{T}"), dev, 32, 100)
                           for T in (32768, 131072)]
    return out


def run_grid(args):
    """(P, K_c) grid of the paper's Table 3 (context 65536) on this build: us per layer, closed form."""
    import torch
    from dataclasses import replace
    from workloads import config_spec
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cells = []
    for P in (8, 16, 32, 64, 96):
        for K_c in (64, 128, 192, 256):
            if K_c > P * 16:
                continue
            spec = replace(config_spec(2, batch=8, T=65536, layers=8), P=P, K_c=K_c,
                           name=f"cfg2_b8_t65536_P{P}_Kc{K_c}")
            p = measure_point(spec, dev, 30, want_kernels=False)
            cells.append({"P": P, "K_c": K_c, "us_per_layer": p["us_per_layer"]})
    spec = config_spec(2, batch=8, T=65536, layers=8, name="cfg2_b8_t65536")
    a = parse_args(["--dense-baseline"])
    h = Harness(spec, dev, args=a)
    step = h.capture(True)
    with torch.cuda.stream(h.stream):
        for _ in range(3):
            step()
    dense_us = h.time_steps(step, 10) / 10 * 1e3 / h.L
    print(json.dumps({"grid": cells, "dense_split_k_us_per_layer": dense_us, "batch": 8, "context": 65536,
                      "unit": "us per layer, graph replay over 8 distinct layer caches"}), flush=True)


def run_leak_curve(args):
    """Leakage against the gap statistic (Sec. 8 / Cor. 1): per unit the proxy gap, its bound, the TRUE
    softmax mass outside the candidate set and the output error (fp64 dense pass), binned by gap / epsilon.
    CPU oracle only."""
    import numpy as np
    import oracle
    from workloads import config_spec, make_workload
    rows = []
    for needles in (0, 1, 2, 4, 8):
        for seed in (0, 1):
            spec = config_spec(0, needles=needles, name=f"cfg0_needles{needles}")
            w = make_workload(spec, seed=0x1EA40000 + 10 * needles + seed)
            geo, q, K, V, bt, sl = oracle_inputs(w)
            st = oracle.decode_step(geo, q, K, V, bt, sl, spec.P, spec.K_c, w.epsilon, w.gap_threshold)
            dn = oracle.dense(geo, q, K, V, bt, sl, w.epsilon, cand_pos=st.sparse.cand_pos)
            err = np.linalg.norm(dn.out - st.sparse.out, axis=-1) / np.maximum(np.linalg.norm(dn.out, axis=-1), 1e-300)
            for g, lb, tl, e in zip(st.sparse.delta.reshape(-1) / w.epsilon, st.sparse.leak_bound.reshape(-1),
                                    dn.true_leak.reshape(-1), err.reshape(-1)):
                rows.append((float(g), float(lb), float(tl), float(e)))
    rows = np.array(rows)
    bins = [(0, 2), (2, 4), (4, 8), (8, 16), (16, 32), (32, np.inf)]
    table = []
    for lo, hi in bins:
        m = (rows[:, 0] >= lo) & (rows[:, 0] < hi)
        if not m.any():
            continue
        r = rows[m]
        table.append({"gap_over_eps": [lo, None if np.isinf(hi) else hi], "units": int(m.sum()),
                      "bound_median": float(np.median(r[:, 1])), "true_leak_median": float(np.median(r[:, 2])),
                      "true_leak_max": float(r[:, 2].max()), "rel_err_median": float(np.median(r[:, 3])),
                      "rel_err_max": float(r[:, 3].max()),
                      "units_leak_above_bound": int((r[:, 2] > r[:, 1] * (1 + 1e-9) + 1e-300).sum())})
    print(json.dumps({"leak_curve": table, "units": int(len(rows)),
                      "workloads": "config 0 shape, 0/1/2/4/8 needles per KV head, two seeds each"}), flush=True)


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2602_13804_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()

    spec = workload_spec(args.workload, args.layers)
    if args.P is not None or args.Kc is not None:      # the (P, K_c) ablation grid of the paper's Table 3
        from dataclasses import replace
        P_new = args.P if args.P is not None else spec.P
        K_new = args.Kc if args.Kc is not None else spec.K_c
        spec = replace(spec, P=P_new, K_c=K_new, name=f"{spec.name}_P{P_new}_Kc{K_new}")
    if args.needle_mode:
        from dataclasses import replace
        spec = replace(spec, needle_mode=args.needle_mode, name=f"{spec.name}_{args.needle_mode}")
    h = Harness(spec, dev, rank=rank, args=args)
    L, distinct, shape, units = h.L, h.distinct, h.shape, h.units
    P, K_c, eps, tau = h.P, h.K_c, h.eps, h.tau
    layers, summaries, stream = h.layers, h.summaries, h.stream
    w0 = layers[0]
    out, diag, routed, flist, fcount, ws = h.out, h.diag, h.routed, h.flist, h.fcount, h.ws
    solve, cert = h.solve, h.cert
    summary_ms = h.summary_ms_per_layer

    kernels_per_layer = 1 if args.dense_baseline else 3   # scan, sparse (top-P selection fused in), dense
    if cert is not None and args.expand:
        kernels_per_layer = 3 + vsa_expand_rounds(P, args.expand)
    if args.two_level:
        kernels_per_layer = 6     # prep, representative scan, super-page selection, inner scan, sparse, dense
    use_graph = not args.no_graph
    step = h.capture(use_graph)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            step()
        barrier()
        sampler = ClockSampler(local)
        sampler.start()
        time.sleep(0.25)
        t_wall0 = time.time()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
        e0.record(stream)
        for k in range(args.steps):
            step()
            marks[k].record(stream)       # per-step spread only; the figure of merit is e0 -> e1
        e1.record(stream)
        barrier()
        ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
        ms_per_step = ms_total / args.steps
        per_step = np.array([a.elapsed_time(b) for a, b in zip([e0] + marks[:-1], marks)])
        step_spread = {"median_ms": float(np.median(per_step)), "p10_ms": float(np.percentile(per_step, 10)),
                       "p90_ms": float(np.percentile(per_step, 90))}
        # The same step, repeated inside one more event pair until that region is long enough for the
        # 100 ms clock sampler to fall inside it: the clock record below describes timed work only.
        n_sus = max(args.steps, int(math.ceil(SUSTAIN_S / max(ms_per_step * 1e-3, 1e-6))))
        n_sus = min(n_sus, 200000)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for _ in range(n_sus):
            step()
        s1.record(stream)
        barrier()
        t_wall1 = time.time()
        sustained_ms_per_step = max_over_ranks(s0.elapsed_time(s1), world, dev) / n_sus
        clocks = sampler.stop(t_wall0, t_wall1)

        # fallback statistics of the last layer that ran
        fb_units = h.fallback_units() if not args.dense_baseline else np.arange(units)
        fb_count = len(fb_units)

        # ---- per-kernel timing of the same launch sequence (events between the kernels) ----
        per_kernel = None
        if not args.dense_baseline:
            per_kernel = h.per_kernel(step, max(3, min(args.steps, 10)))

        # ---- with --solver-iters / --certified: the closed-form step timed the same way ----
        closed_form_us_per_layer = None
        if solve is not None or cert is not None or args.two_level or args.group_shared:
            step_c = h.capture(use_graph, plain=True)
            for _ in range(3):
                step_c()
            barrier()
            closed_form_us_per_layer = h.time_steps(step_c, args.steps, world, barrier) / args.steps * 1e3 / L

        # ---- end to end: q from pinned host memory, out + diag back to the host, every layer ----
        e2e = None
        if not args.dense_baseline and solve is None and cert is None and not args.two_level and \
                not args.group_shared:
            q_host = [w.q.cpu().pin_memory() for w in layers]
            q_dev = torch.empty_like(w0.q)
            out_host = torch.empty(out.shape, dtype=torch.float32).pin_memory()
            diag_host = torch.empty((units, B.DIAG_BYTES // 4), dtype=torch.int32).pin_memory()

            def enqueue_e2e():
                for i in range(L):
                    w, s = layers[i % distinct], summaries[i % distinct]
                    B.vsa_decode_step_host(shape, q_host[i % distinct], q_dev, s, w.k_cache, w.v_cache, w.block_table,
                                           w.seq_lens, P, K_c, eps, tau, out_host, out, diag_host, diag, routed,
                                           flist, fcount, ws)

            # the same API calls captured once (copies from and to the pinned buffers become graph
            # nodes; a replay reads whatever the host has put into q_host by then)
            graph_e2e = None
            if use_graph:
                enqueue_e2e()
                stream.synchronize()
                graph_e2e = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph_e2e, stream=stream):
                    enqueue_e2e()

            def step_e2e():
                if graph_e2e is not None:
                    graph_e2e.replay()
                else:
                    enqueue_e2e()
                stream.synchronize()      # the host reads the step's result

            for _ in range(3):
                step_e2e()
            barrier()
            e0.record(stream)
            for _ in range(args.steps):
                step_e2e()
            e1.record(stream)
            barrier()
            ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
            h2d = L * units * 128 * 2
            d2h = L * units * (128 * 4 + B.DIAG_BYTES)
            e2e = {"value": us_per_token_per_layer(ms_e2e, world, shape.batch, L), "unit": UNIT, "ms_per_step": ms_e2e,
                   "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                   "api": "vsa_decode_step_host per layer, " +
                          ("captured in a CUDA graph" if graph_e2e is not None else "plain stream launches") +
                          ", one stream sync per step"}

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- the oracle on one layer: CPU baseline, and the routed / candidate sets for the byte model ----
    last = layers[(L - 1) % distinct]        # the layer whose fallback list is in the buffers
    sl = w0.seq_lens.cpu().numpy().astype(np.int64)
    cpu_baseline = None
    rp = cp = None
    run_oracle = not args.no_cpu_baseline and world == 1 and not args.dense_baseline
    if run_oracle:
        import oracle
        inputs = oracle_inputs(last)
        geo, q_, K_, V_, bt_, sl_ = inputs
        st = oracle.decode_step(geo, q_, K_, V_, bt_, sl_, P, K_c, eps, tau)
        rp, cp = st.route.pages, st.sparse.cand_pos
        sec, reps, cores = oracle_layer_time(last, inputs=inputs)
        cpu_baseline = {"value": sec * 1e6 / shape.batch, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"one layer of {L}, all {shape.batch} sequences, {reps} repetitions of one "
                                  f"oracle decode step (summaries prebuilt)"}
        # the same oracle step on one thread, and the oracle's dense definition on all threads, a few
        # repetitions each (context for the figure above, same unit)
        oracle.set_num_threads(1)
        sec1, reps1, _ = oracle_layer_time(last, reps_budget_s=4.0, inputs=inputs)
        oracle.set_num_threads(cores)
        secd, repsd, _ = oracle_layer_time(last, reps_budget_s=4.0, dense=True, inputs=inputs)
        cpu_baseline["single_thread_value"] = sec1 * 1e6 / shape.batch
        cpu_baseline["dense_definition_value"] = secd * 1e6 / shape.batch
        cpu_baseline["extra_samples"] = f"{reps1} single-thread repetitions, {repsd} dense repetitions of the same layer"

    # ---- algorithmic bytes per launch and the roofline fractions ----
    fallback = np.zeros(units, np.int32)
    fallback[fb_units] = 1
    alg = algorithmic_bytes(spec, sl, rp, cp, fallback)
    peak, peak_kind = measured_peak()
    step_us = ms_per_step * 1e3 / L
    if args.dense_baseline:
        kern = {"dense_fallback": {"bytes_per_launch": alg["dense_fallback"], "us_per_launch": step_us}}
        g = alg["dense_fallback"] / (step_us * 1e-6) / 1e9
        kern["dense_fallback"].update({"achieved_GBps": g, "frac": g / peak, "frac_of_8TBps": g / NOMINAL_HBM_GBS})
        dom = "dense_fallback"
    else:
        kern = kernel_fracs(alg, per_kernel, step_us, peak)
        dom = max(("route_scan", "sparse_decode", "dense_fallback"), key=lambda k: per_kernel[k])
        if solve is not None or cert is not None or args.two_level or args.group_shared:
            # the events bracket the plain step's kernels; the cost of the iterations (of the certificate)
            # is the difference of the two graph-replayed steps and is booked on the sparse kernel
            extra = step_us - closed_form_us_per_layer
            dom = "sparse_decode"
            k = kern[dom]
            k["us_solver_iterations"] = extra
            k["us_per_launch"] += extra
            k["achieved_GBps"] = k["bytes_per_launch"] / (k["us_per_launch"] * 1e-6) / 1e9
            k["frac"], k["frac_of_8TBps"] = k["achieved_GBps"] / peak, k["achieved_GBps"] / NOMINAL_HBM_GBS
    d = kern[dom]
    traffic = ncu_traffic(dom, spec.name)
    roofline = {"bound": "hbm", "achieved": d["achieved_GBps"], "peak": peak, "unit": "GB/s", "frac": d["frac"],
                "traffic": traffic, "kernel": dom, "bytes_per_launch": d["bytes_per_launch"],
                "us_per_launch": d["us_per_launch"], "peak_kind": f"of {peak_kind}",
                "frac_of_8TBps": d["frac_of_8TBps"],
                "bytes_model": "union over each GQA group of routed K pages and candidate V rows (oracle sets of "
                               "one layer)" if "sparse_union_pages" in alg else "per kernel, see `kernels`",
                "us_is": "CUDA-event interval around the kernel inside vsa_decode_step_timed; nothing subtracted",
                "us_event_pair_overhead": per_kernel["event_pair_overhead"] if per_kernel else None,
                "frac_traffic_based": (traffic / (d["us_per_launch"] * 1e-6) / 1e9 / peak) if traffic else None}
    if "frac_per_head_model" in d:
        roofline["frac_per_head_model"] = d["frac_per_head_model"]
    if "sparse_union_pages" in alg:
        roofline["union_pages"], roofline["union_rows"] = alg["sparse_union_pages"], alg["sparse_union_rows"]
    # the second ceiling of a kernel that is not limited by bytes: warp instructions issued (one ncu capture,
    # profiles/ncu_traffic.txt) against the SMs' issue slots, 4 schedulers per SM at the sampled SM clock
    inst = ncu_traffic(dom + "_warp_instructions", spec.name)
    if inst and clocks.get("sm_mhz"):
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        issue_peak = sms * 4 * clocks["sm_mhz"] * 1e6
        roofline["issue_slots"] = {"warp_instructions_per_launch": inst, "peak_per_s": issue_peak,
                                   "frac": inst / (d["us_per_launch"] * 1e-6) / issue_peak,
                                   "note": "neither ceiling is approached: the kernel is a chain of dependent phases "
                                           "(two exact selections, two dependent gathers) bound by latency"}

    sweep_obj = None
    default_run = (args.workload == "cfg1" and not args.dense_baseline and solve is None and cert is None
                   and args.P is None and args.Kc is None and args.layers is None and not args.two_level
                   and not args.group_shared and not args.needle_mode)
    if default_run and world == 1 and not args.no_sweep:
        h.release()
        del layers, summaries, w0, last, h
        torch.cuda.empty_cache()
        sweep_obj = sweep(dev)

    value = us_per_token_per_layer(ms_per_step, world, shape.batch, L)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": spec.name, "batch": shape.batch, "n_q_heads": shape.n_q_heads,
                   "n_kv_heads": shape.n_kv_heads, "head_dim": 128, "page_size": spec.page_size,
                   "context": int(sl.max()), "P": P, "K_c": K_c, "epsilon": eps, "gap_threshold": tau,
                   "layers_per_step": L, "distinct_layer_caches": distinct,
                   "l2": f"inputs larger than L2: {distinct} distinct layer caches, "
                         f"{(alg['route_scan'] + alg.get('sparse_decode', alg['sparse_decode_per_head_model'])) * distinct / 1e6:.0f}"
                         f" MB touched per pass over them",
                   "launch": "cuda graph replay of the whole step" if use_graph else "plain stream launches",
                   "path": "dense split-K baseline" if args.dense_baseline else
                           ("route -> group-shared sparse (one page set and one candidate set per KV head) -> "
                            "dense fallback" if args.group_shared else
                            f"two-level route ({args.two_level} super-pages per unit) -> sparse -> dense fallback"
                            if args.two_level else
                            (f"route -> sparse with routing certificate -> retries of the refused units with up to "
                             f"{args.expand} pages -> dense fallback") if cert is not None and args.expand else
                            "route -> sparse with routing certificate -> dense fallback" if cert is not None else
                            "route -> sparse -> dense fallback" if solve is None else
                            f"route -> sparse with {args.solver_iters} " +
                            ("Frank-Wolfe" if args.solver == "fw" else "entropic mirror-descent") +
                            " iterations -> dense fallback")},
        "latency_us_per_layer": step_us,
        "step_spread": step_spread,
        "sustained": {"steps": n_sus, "ms_per_step": sustained_ms_per_step,
                      "note": "the same step repeated inside one event pair; the clock samples come from the "
                              "timed and the sustained region"},
        "per_kernel_us": per_kernel, "kernels": kern, "closed_form_latency_us_per_layer": closed_form_us_per_layer,
        "fallback_fraction_last_layer": fb_count / units,
        "summary_build_ms_per_layer": summary_ms,
        "gpu_launches": args.steps * L * kernels_per_layer, "clocks": clocks, "e2e": e2e, "roofline": roofline,
        "cpu_baseline": cpu_baseline, "sweep": sweep_obj,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def vsa_expand_rounds(P: int, P_max: int) -> int:
    """Launches of the fused kernel the expanding step adds: one per doubling of P up to P_max."""
    n, p = 0, P
    while p < P_max:
        p = min(2 * p, P_max)
        n += 1
    return n


def ncu_traffic(kernel: str, workload: str):
    """DRAM bytes per launch of `kernel` on `workload` as captured once with ncu, or None.
    profiles/ncu_traffic.txt holds lines `workload kernel dram_bytes_per_launch`."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    try:
        with open(path) as f:
            for ln in f:
                parts = ln.split()
                if len(parts) >= 3 and not ln.startswith("#") and parts[0] == workload and parts[1] == kernel:
                    return float(parts[2])
    except Exception:
        pass
    return None


def main():
    args = parse_args()
    if args.leak_curve:
        return run_leak_curve(args)
    if args.fp8:
        import torch
        dev = torch.device("cuda", 0)
        torch.cuda.set_device(dev)
        print(json.dumps(fp8_point(workload_spec(args.workload, args.layers), dev, args.steps)))
        return
    if args.impl == "reference" and "WORLD_SIZE" not in os.environ:
        return run_reference(args)           # one process: the oracle runs on this host's cores
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # start the N ranks (one process per GPU); their rank 0 prints the JSON line
        cmd = spawn_command(sys.argv[1:], args.gpus, free_port())
        sys.exit(subprocess.call(cmd))
    if args.impl == "reference":
        run_reference(args)
    elif args.grid:
        run_grid(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
