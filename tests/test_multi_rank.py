"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own forest, no data-path collective."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from conftest import ROOT


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import schedule as osched
    w = bench.rank_workload(1, rank)
    f = w.forest
    depth, level_ptr, perm, _, n_levels = osched.schedule(f.child_ptr, f.child_idx, f.n_nodes)
    # the slowest rank's time and the sum of nodes, as bench.py reduces them
    t, n = bench.job_totals(0.5 + rank, f.n_nodes, world, torch.device("cpu"))
    out[rank] = (f.n_nodes, int(f.child_idx.sum()), n_levels, t, n)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_draw_different_forests_and_reduce_totals():
    world = 2
    port = 29500 + os.getpid() % 2000
    manager = mp.Manager()
    out = manager.dict()
    mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
    (n0, sig0, l0, t0, tot0), (n1, sig1, l1, t1, tot1) = out[0], out[1]
    assert (n0, sig0) != (n1, sig1)            # different seeds, same shape
    assert abs(n0 - n1) < 0.5 * n0
    assert t0 == t1 == 1.5                      # max over ranks
    assert tot0 == tot1 == float(n0 + n1)       # whole-job node count


def test_rank_zero_matches_the_single_gpu_workload():
    import bench
    from paper_1904_07421_b200 import workloads as wl
    a, b = bench.rank_workload(2, 0), wl.make_workload(2)
    assert np.array_equal(a.forest.child_idx, b.forest.child_idx) and np.array_equal(a.token, b.token)


def test_bench_starts_its_own_ranks_when_launched_bare():
    """`python bench.py --gpus 2` without WORLD_SIZE re-launches itself as two ranks on 127.0.0.1; with
    --rendezvous-only the ranks meet over gloo on the CPU, reduce the totals like the timed path does, and rank 0
    prints one line that says n_gpus = 2."""
    import json
    import subprocess
    import bench
    cmd = bench.launcher_command(2, ["--gpus", "2", "--rendezvous-only"], 29400)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rendezvous-only"],
                         capture_output=True, text=True, timeout=240, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    n0 = bench.rank_workload(1, 0).forest.n_nodes
    n1 = bench.rank_workload(1, 1).forest.n_nodes
    assert out["n_gpus"] == 2 and out["max_seconds"] == 2.0 and out["total_nodes"] == float(n0 + n1)
