"""The N > 1 path on CPU: two gloo ranks.  The decode step shards by sequence with no exchange of
data, so (1) each rank working on its own sequences reproduces exactly what one process computes on
the whole batch, and (2) the only cross-rank host logic is the timing reduction (slowest rank) and
the whole-job metric; the reference arm of the benchmark runs on rank 0 only."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from util import bits
from workloads import WorkloadSpec, make_workload

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spec():
    return WorkloadSpec(name="mp", config=6, batch=4, n_q_heads=8, n_kv_heads=2, P=6, K_c=40,
                        seq_lens=(900, 333, 1500, 64), needles=3)


def _oracle_on(w, rows):
    geo = oracle.Geometry(batch=len(rows), n_q_heads=8, n_kv_heads=2, max_pages_per_seq=w.max_pages_per_seq,
                          num_pool_pages=w.pool_pages)
    return oracle.decode_step(geo, bits(w.q[rows]), bits(w.k_cache), bits(w.v_cache),
                              w.block_table[rows].numpy(), w.seq_lens[rows].numpy(), 6, 40, w.epsilon,
                              w.gap_threshold)


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = make_workload(_spec(), seed=606)                 # same cache on every rank, sharded by sequence
        rows = list(range(rank * 2, rank * 2 + 2))
        st = _oracle_on(w, rows)
        # gather the shards' results on rank 0: no data-path collective is needed to PRODUCE them
        mine = torch.from_numpy(np.concatenate([st.out.reshape(2, -1), st.sparse.fallback.reshape(2, -1).astype(np.float64),
                                                st.route.pages.reshape(2, -1).astype(np.float64)], axis=1))
        gathered = [torch.empty_like(mine) for _ in range(world)] if rank == 0 else None
        dist.gather(mine, gathered, dst=0)
        # timing reduction: the step takes as long as the slowest rank
        slowest = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
        assert slowest == 15.0
        assert bench.us_per_token_per_layer(slowest, world, 2, 32) == pytest.approx(15.0e3 / (2 * 2 * 32))
        if rank == 0:
            np.save(os.path.join(out_dir, "gathered.npy"), torch.cat(gathered).numpy())
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_sharded_by_sequence_reproduce_the_single_process_result(tmp_path):
    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    got = np.load(os.path.join(str(tmp_path), "gathered.npy"))
    w = make_workload(_spec(), seed=606)
    full = _oracle_on(w, [0, 1, 2, 3])
    want = np.concatenate([full.out.reshape(4, -1), full.sparse.fallback.reshape(4, -1).astype(np.float64),
                           full.route.pages.reshape(4, -1).astype(np.float64)], axis=1)
    assert np.array_equal(got, want)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg0",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg0",
                        "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0
    import json
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["higher_is_better"] is False


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus N` without a torchrun environment re-launches itself as N ranks.  The launch line
    is exercised here with the reference arm as the CPU stand-in for the ranks' work: two processes start,
    rank 0 prints the one JSON line with n_gpus = 2, rank 1 prints nothing, and the launcher exits 0."""
    sys.path.insert(0, ROOT)
    import bench
    import json
    cmd = bench.spawn_command(["--impl", "reference", "--workload", "cfg0", "--steps", "1", "--warmup", "0",
                               "--gpus", "2"], 2, _free_port())
    assert "torch.distributed.run" in cmd and "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2


def test_expand_round_count():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.vsa_expand_rounds(32, 64) == 1 and bench.vsa_expand_rounds(32, 128) == 2
    assert bench.vsa_expand_rounds(16, 100) == 3 and bench.vsa_expand_rounds(32, 32) == 0
