"""The N > 1 logic of bench.py on CPU: two gloo ranks (replicas only: no data-path collective,
the only exchange is the max over ranks of the measured time), and the reference arm under
torchrun, where rank 0 alone works and prints."""

from __future__ import annotations

import json
import os
import subprocess
import sys

import pytest


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)            # rank 1 is the slow replica
    # coordinate shards: each rank builds its own slice from (rank, world); the slices tile p
    from workloads import build_config, shard_coordinates
    wl = build_config("quad_tree64", seed=0, n=8, p=1001, K=4)
    lo, hi = shard_coordinates(wl, rank, world).meta["coordinates"]
    import torch
    spans = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(spans, torch.tensor([lo, hi]))
    assert spans[0][0] == 0 and spans[-1][1] == wl.p and all(int(a[1]) == int(b[0]) for a, b in zip(spans, spans[1:]))
    out.put((rank, ms, bench.whole_job_rate(1000, world, ms * 1e-3)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_max_time_and_aggregate_rate():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for rank, ms, rate in got:
        assert ms == 15.0                                    # the max, on every rank
        assert abs(rate - 2 * 1000 / 0.015) < 1e-6           # whole job: both replicas' units / slowest time


def test_single_process_helpers_need_no_process_group():
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_rate(10, 1, 2.0) == 5.0


def test_reference_arm_under_torchrun_rank0_only(repo_root):
    port = 31500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), "bench.py", "--impl", "reference",
           "--gpus", "2", "--config", "ls_ring4", "--steps", "1", "--warmup", "1"]
    r = subprocess.run(cmd, cwd=repo_root, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # the other rank exits 0 without work
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "node_activations_per_s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["n_gpus"] == 2 and d["config"]["workload"] == "ls_ring4"


def test_gpus_flag_without_its_ranks_is_refused(repo_root):
    """`--gpus 8` started as one plain process must not print an n_gpus = 1 line: it exits
    non-zero and says how to launch the ranks."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, "bench.py", "--gpus", "8", "--steps", "1"], cwd=repo_root, env=env,
                       capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "torch.distributed.run" in r.stderr
    assert not any(ln.startswith("{") for ln in r.stdout.splitlines())
