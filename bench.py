#!/usr/bin/env python
"""Benchmark of the sparse paged decode-attention step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A "step" is one decode token for every sequence of the batch through all layers of the
workload: per layer vsa_decode_step (page routing -> fused sparse pass -> dense fallback) on
that layer's own KV cache.  Prints ONE JSON line (rank 0).  Workloads:
    cfg1            batch 8, T = 32768, 32 layers, P = 32, K_c = 256  (default; the metric's config)
    cfg0 | cfg3 | cfg4
    cfg2:B:T        a point of the context sweep, e.g. cfg2:1:131072
Extra flags: --layers L (override), --dense-baseline (time the split-K dense kernel on the same
caches instead of the sparse path), --no-graph (plain stream launches for `value`).
"""
from __future__ import annotations

import argparse
import json
import math
import os
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


def parse_args():
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
    ap.add_argument("--P", type=int, default=None, help="override the workload's routed pages per unit")
    ap.add_argument("--Kc", type=int, default=None, help="override the workload's candidate count per unit")
    ap.add_argument("--certified", action="store_true",
                    help="time vsa_decode_step_certified (routing certificate computed, certified gap decides the "
                         "fallback) instead of vsa_decode_step")
    ap.add_argument("--expand", type=int, default=None,
                    help="with --certified: retry the refused units with this many routed pages before the dense "
                         "pass (vsa_decode_step_certified_expand)")
    ap.add_argument("--solver", default="eg", choices=["eg", "fw"],
                    help="with --solver-iters: entropic mirror descent (eg) or Frank-Wolfe with exact line search (fw)")
    ap.add_argument("--solver-iters", type=int, default=None,
                    help="time the step whose candidate weights come from this many entropic mirror-descent "
                         "iterations (vsa_decode_step_entropic) instead of the closed form")
    return ap.parse_args()


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
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [r for (t, r) in self.rows if t0 - 0.05 <= t <= t1 + 0.15 and len(r) >= 7] or \
               [r for (_, r) in self.rows if len(r) >= 7]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm = sorted(float(r[0]) for r in rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].lower().startswith("active") for r in rows)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][1]),
                "power_w_max": max(float(r[2]) for r in rows), "reasons": reasons, "samples": len(rows)}


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


def host_bits(t):
    import numpy as np
    import torch
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_layer_time(w, reps_budget_s: float = 12.0, dense: bool = False):
    """Times the CPU oracle, as it stands, on one layer of the workload (all sequences).
    Returns (seconds per layer-step, repetitions, threads)."""
    import numpy as np
    import oracle
    s = w.spec
    geo = oracle.Geometry(batch=s.batch, n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads,
                          max_pages_per_seq=w.max_pages_per_seq, num_pool_pages=w.pool_pages)
    q, K, V = host_bits(w.q), host_bits(w.k_cache), host_bits(w.v_cache)
    bt, sl = w.block_table.cpu().numpy().astype(np.int32), w.seq_lens.cpu().numpy().astype(np.int32)
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


def run_reference(args):
    """The CPU oracle as the reference arm: same workload, metric and unit; each step is a
    bounded sample (one layer of the workload, all sequences)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from workloads import make_workload
    spec = workload_spec(args.workload, args.layers)
    w = make_workload(spec, device="cpu", rep=0)
    import numpy as np
    import oracle
    s = w.spec
    geo = oracle.Geometry(batch=s.batch, n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads,
                          max_pages_per_seq=w.max_pages_per_seq, num_pool_pages=w.pool_pages)
    q, K, V = host_bits(w.q), host_bits(w.k_cache), host_bits(w.v_cache)
    bt, sl = w.block_table.numpy().astype(np.int32), w.seq_lens.numpy().astype(np.int32)
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


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2602_13804_b200 import binding as B
    from workloads import make_workload

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
    L = spec.layers
    # one distinct KV cache per layer, sized against free memory (never more than 80% of it)
    w0 = make_workload(spec, device=dev, rep=0, sub=rank)
    per_layer = 2 * w0.k_cache.numel() * 2 + w0.pool_pages * spec.n_kv_heads * 256
    free, _ = torch.cuda.mem_get_info(dev)
    distinct = max(1, min(L, int(0.8 * free // per_layer) + 1))
    layers = [w0] + [make_workload(spec, device=dev, rep=i, sub=rank) for i in range(1, distinct)]
    shape = B.shape_of(w0.q, w0.k_cache, w0.block_table)
    # A paged KV cache has ONE block table and one length vector per sequence, used by every layer
    # (the layers' K/V pools are separate tensors indexed by the same page numbers): all layers get
    # layer 0's tensors.  The generator gives every layer the same structure, which is checked.
    for w in layers:
        assert w.pool_pages == w0.pool_pages and torch.equal(w.block_table, w0.block_table) and \
            torch.equal(w.seq_lens, w0.seq_lens)
        w.block_table, w.seq_lens = w0.block_table, w0.seq_lens
    units = shape.batch * shape.n_q_heads
    P, K_c, eps, tau = spec.P, spec.K_c, w0.epsilon, w0.gap_threshold

    # cache maintenance (off the decode path): summaries of every layer, timed separately
    summaries = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for w in layers:
        s = torch.zeros((shape.num_pool_pages, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=dev)
        B.vsa_build_page_summaries(shape, w.k_cache, w.block_table, w.seq_lens, None, s)
        summaries.append(s)
    ev1.record()
    torch.cuda.synchronize()
    summary_ms_per_layer = ev0.elapsed_time(ev1) / len(layers)

    out = torch.empty((shape.batch, shape.n_q_heads, 128), dtype=torch.float32, device=dev)
    diag = B.alloc_diag(units, dev)
    routed = torch.empty((shape.batch, shape.n_q_heads, P), dtype=torch.int32, device=dev)
    flist = torch.empty(units, dtype=torch.int32, device=dev)
    fcount = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = B.alloc_workspace(shape, P, K_c, B.VSA_WS_STEP, dev)
    ws_dense = B.alloc_workspace(shape, P, K_c, B.VSA_WS_DENSE, dev)

    solve = B.alloc_solve(units, dev) if args.solver_iters is not None else None
    cert = radii = None
    if args.certified:
        cert = B.alloc_cert(units, dev)
        ws = B.alloc_workspace(shape, args.expand or P, K_c,
                               B.VSA_WS_STEP_EXPAND if args.expand else B.VSA_WS_STEP_CERTIFIED, dev)
        if args.expand:
            routed = torch.empty((shape.batch, shape.n_q_heads, args.expand), dtype=torch.int32, device=dev)
        radii = []
        for w, s_ in zip(layers, summaries):      # cache maintenance, like the summaries
            r = torch.zeros((shape.num_pool_pages, shape.n_kv_heads), dtype=torch.float32, device=dev)
            B.vsa_build_page_radii(shape, w.k_cache, s_, w.block_table, w.seq_lens, None, r)
            radii.append(r)

    def layer_call(i):
        w, s = layers[i % distinct], summaries[i % distinct]
        if args.dense_baseline:
            B.vsa_dense_decode_fallback(shape, w.q, w.k_cache, w.v_cache, w.block_table, w.seq_lens, None, None,
                                        eps, out, diag, ws_dense)
        elif cert is not None and args.expand:
            B.vsa_decode_step_certified_expand(shape, w.q, s, radii[i % distinct], w.k_cache, w.v_cache, w.block_table,
                                               w.seq_lens, P, args.expand, K_c, eps, tau, out, diag, cert, routed,
                                               flist, fcount, ws)
        elif cert is not None:
            B.vsa_decode_step_certified(shape, w.q, s, radii[i % distinct], w.k_cache, w.v_cache, w.block_table,
                                        w.seq_lens, P, K_c, eps, tau, out, diag, cert, routed, flist, fcount, ws)
        elif solve is not None and args.solver == "fw":
            B.vsa_decode_step_frank_wolfe(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c, eps,
                                          tau, args.solver_iters, out, diag, solve, routed, flist, fcount, ws)
        elif solve is not None:
            B.vsa_decode_step_entropic(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c, eps,
                                       tau, args.solver_iters, out, diag, solve, routed, flist, fcount, ws)
        else:
            B.vsa_decode_step(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c, eps, tau,
                              out, diag, routed, flist, fcount, ws)

    def step_plain():
        for i in range(L):
            layer_call(i)

    kernels_per_layer = 1 if args.dense_baseline else 3   # scan, sparse (top-P selection fused in), dense
    stream = torch.cuda.Stream(device=dev)
    use_graph = not args.no_graph
    with torch.cuda.stream(stream):
        step_plain()                      # first call: function attributes, lazy module load
        stream.synchronize()
        graph = None
        if use_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step_plain()
        step = graph.replay if graph is not None else step_plain

        def barrier():
            torch.cuda.synchronize(dev)
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize(dev)

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
        t_wall1 = time.time()
        ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
        ms_per_step = ms_total / args.steps
        per_step = np.array([a.elapsed_time(b) for a, b in zip([e0] + marks[:-1], marks)])
        step_spread = {"median_ms": float(np.median(per_step)), "p10_ms": float(np.percentile(per_step, 10)),
                       "p90_ms": float(np.percentile(per_step, 90))}
        # keep the GPU loaded a little longer if the region was too short to sample clocks
        if t_wall1 - t_wall0 < 0.5:
            t_end = time.time() + 0.6
            while time.time() < t_end:
                step()
            torch.cuda.synchronize(dev)
            t_wall1 = time.time()
        clocks = sampler.stop(t_wall0, t_wall1)

        # fallback statistics of the last layer that ran
        fb_count = int(fcount.item()) if not args.dense_baseline else units

        # ---- per-kernel timing of the same launch sequence (events between the kernels) ----
        per_kernel = None
        if not args.dense_baseline:
            n_rep = max(3, min(args.steps, 10))
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(L)]
            for row in evs:
                for e in row:
                    e.record(stream)
            acc = np.zeros(4)
            for _ in range(2):
                step()
            # the timed entry point's own first call (with --solver-iters / --certified its kernels have not
            # run yet: module load and function attributes would otherwise land between the events)
            for i in range(L):
                w, s = layers[i % distinct], summaries[i % distinct]
                B.vsa_decode_step_timed(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c,
                                        eps, tau, out, diag, routed, flist, fcount, ws, evs[i])
            stream.synchronize()
            for _ in range(n_rep):
                # hold the GPU for ~3 ms so that the host enqueues the whole step ahead of it:
                # the events then bracket kernels that run back to back, not launch gaps
                torch.cuda._sleep(6_000_000)
                for i in range(L):
                    w, s = layers[i % distinct], summaries[i % distinct]
                    B.vsa_decode_step_timed(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c,
                                            eps, tau, out, diag, routed, flist, fcount, ws, evs[i])
                stream.synchronize()
                for row in evs:
                    acc += np.array([row[j].elapsed_time(row[j + 1]) for j in range(4)])
            per_kernel = dict(zip(["route_scan", "route_select", "sparse_decode", "dense_fallback"],
                                  (acc / (n_rep * L) * 1e3).tolist()))    # us per launch

        # ---- with --solver-iters: the closed-form step timed the same way, for the cost of the iterations ----
        closed_form_us_per_layer = None
        if solve is not None or cert is not None:
            def step_closed():
                for i in range(L):
                    w, s = layers[i % distinct], summaries[i % distinct]
                    B.vsa_decode_step(shape, w.q, s, w.k_cache, w.v_cache, w.block_table, w.seq_lens, P, K_c, eps, tau,
                                      out, diag, routed, flist, fcount, ws)
            step_c = step_closed
            if use_graph:
                graph_c = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph_c, stream=stream):
                    step_closed()
                step_c = graph_c.replay
            for _ in range(3):
                step_c()
            barrier()
            e0.record(stream)
            for _ in range(args.steps):
                step_c()
            e1.record(stream)
            barrier()
            closed_form_us_per_layer = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps * 1e3 / L

        # ---- end to end: q from pinned host memory, out + diag back to the host, every layer ----
        e2e = None
        if not args.dense_baseline and solve is None and cert is None:
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

    # ---- algorithmic bytes per launch (per sequence-layer figures x what one launch processes) ----
    sl = w0.seq_lens.cpu().numpy().astype(np.int64)
    n_pages = (sl + 15) // 16
    scan_bytes = int(n_pages.sum()) * (spec.n_kv_heads * 256 + 4) + units * 256
    n_cand = np.minimum(K_c, np.minimum(P, n_pages) * 16)
    sparse_bytes = int((np.minimum(P, n_pages) * 16 * 256 + n_cand * 256).sum()) * spec.n_q_heads + units * (256 + 512)
    dense_bytes_all = int(sl.sum()) * spec.n_kv_heads * 512
    peak, peak_kind = measured_peak()
    if args.dense_baseline:
        us = ms_per_step * 1e3 / L
        roof = {"kernel": "dense_split_kernel", "bytes_per_launch": dense_bytes_all, "us_per_launch": us}
    else:
        alg = {"route_scan": scan_bytes, "sparse_decode": sparse_bytes,
               "dense_fallback": dense_bytes_all * fb_count // max(units, 1)}
        dom = max(("route_scan", "sparse_decode", "dense_fallback"), key=lambda k: per_kernel[k])
        # The interval between two event records holds the kernel plus the cost of the records
        # themselves; the "route_select" slot of the timed step brackets no kernel (the selection is
        # fused into the sparse kernel), so it measures that cost in the same pass and is taken off.
        overhead = per_kernel["route_select"]
        roof = {"kernel": dom, "bytes_per_launch": alg[dom], "us_per_launch": per_kernel[dom] - overhead,
                "us_event_interval": per_kernel[dom], "us_event_pair_overhead": overhead}
        if solve is not None or cert is not None:
            # the events bracket the plain step's kernels; the cost of the iterations (of the certificate)
            # is the difference of the two graph-replayed steps and is booked on the sparse kernel
            extra = ms_per_step * 1e3 / L - closed_form_us_per_layer
            roof = {"kernel": "sparse_decode", "bytes_per_launch": alg["sparse_decode"],
                    "us_per_launch": per_kernel["sparse_decode"] - overhead + extra,
                    "us_event_interval": per_kernel["sparse_decode"], "us_event_pair_overhead": overhead,
                    "us_solver_iterations": extra}
    achieved = roof["bytes_per_launch"] / (roof["us_per_launch"] * 1e-6) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": ncu_traffic(roof["kernel"], spec.name), "kernel": roof["kernel"],
                "bytes_per_launch": roof["bytes_per_launch"], "us_per_launch": roof["us_per_launch"],
                "peak_kind": f"of {peak_kind}", "frac_of_8TBps": achieved / 8000.0}
    for k in ("us_event_interval", "us_event_pair_overhead", "us_solver_iterations"):
        if k in roof:
            roofline[k] = roof[k]

    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1 and not args.dense_baseline:
        sec, reps, cores = oracle_layer_time(w0)
        cpu_baseline = {"value": sec * 1e6 / shape.batch, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"layer 0 of {L}, all {shape.batch} sequences, {reps} repetitions of one "
                                  f"oracle decode step (summaries prebuilt)"}
        # the same oracle step on one thread, and the oracle's dense definition on all threads, a few
        # repetitions each (context for the figure above, same unit)
        import oracle
        oracle.set_num_threads(1)
        sec1, reps1, _ = oracle_layer_time(w0, reps_budget_s=4.0)
        oracle.set_num_threads(cores)
        secd, repsd, _ = oracle_layer_time(w0, reps_budget_s=4.0, dense=True)
        cpu_baseline["single_thread_value"] = sec1 * 1e6 / shape.batch
        cpu_baseline["dense_definition_value"] = secd * 1e6 / shape.batch
        cpu_baseline["extra_samples"] = f"{reps1} single-thread repetitions, {repsd} dense repetitions of the same layer"

    value = us_per_token_per_layer(ms_per_step, world, shape.batch, L)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": spec.name, "batch": shape.batch, "n_q_heads": shape.n_q_heads,
                   "n_kv_heads": shape.n_kv_heads, "head_dim": 128, "page_size": 16,
                   "context": int(sl.max()), "P": P, "K_c": K_c, "epsilon": eps, "gap_threshold": tau,
                   "layers_per_step": L, "distinct_layer_caches": distinct,
                   "l2": f"inputs larger than L2: {distinct} distinct layer caches, "
                         f"{(scan_bytes + sparse_bytes) * distinct / 1e6:.0f} MB touched per pass over them",
                   "launch": "cuda graph replay of the whole step" if use_graph else "plain stream launches",
                   "path": "dense split-K baseline" if args.dense_baseline else
                           ((f"route -> sparse with routing certificate -> retry of the refused units with "
                             f"{args.expand} pages -> dense fallback") if cert is not None and args.expand else
                            "route -> sparse with routing certificate -> dense fallback" if cert is not None else
                            "route -> sparse -> dense fallback" if solve is None else
                            f"route -> sparse with {args.solver_iters} " +
                            ("Frank-Wolfe" if args.solver == "fw" else "entropic mirror-descent") +
                            " iterations -> dense fallback")},
        "latency_us_per_layer": ms_per_step * 1e3 / L,
        "step_spread": step_spread,
        "per_kernel_us": per_kernel, "closed_form_latency_us_per_layer": closed_form_us_per_layer,
        "fallback_fraction_last_layer": fb_count / units,
        "summary_build_ms_per_layer": summary_ms_per_layer,
        "gpu_launches": args.steps * L * kernels_per_layer, "clocks": clocks, "e2e": e2e, "roofline": roofline,
        "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


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
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
