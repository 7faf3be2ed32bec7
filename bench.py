"""Benchmark of the batched Tree-LSTM hot path: one step = batching analysis + forward over one forest.

    python bench.py --gpus N --steps K --warmup W [--config 1..5] [--impl reference]

With N > 1 and no WORLD_SIZE in the environment the script starts its N ranks itself (torch.distributed.run on
127.0.0.1); under torchrun it is one of the ranks.  Prints ONE JSON line (rank 0).  Inputs are seeded synthetic forests (workloads.py).  `value` is nodes/s
with inputs resident in HBM; `e2e` is the same step through the host-buffer entry point with the copies
inside the timed region.  At N > 1 every rank runs its own forest of the same shape (trees are
independent: no collective on the data path) and the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1904_07421_b200 import workloads as wl  # noqa: E402

METRIC = "treelstm_forward_nodes_per_sec"
UNIT = "nodes/s"
L2_FLUSH_BYTES = 256 << 20
# fp32 FMA peak of the CUDA cores: 148 SMs x 128 lanes x 2 flops x 1.965 GHz (the part's maximum SM clock)
FP32_ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------------------------------
# reference arm / CPU baseline: the fp64 per-node checker, as it stands, on the host cores
# --------------------------------------------------------------------------------------------------
def oracle_sample(w: wl.Workload, n_trees: int):
    trees = np.arange(min(n_trees, w.forest.n_trees))
    sub, nodes = wl.subforest(w.forest, trees)
    return sub, w.x_rows(nodes)


def oracle_step(w, sub, x):
    from oracle import schedule as osched
    from oracle import treelstm as ot
    osched.schedule(sub.child_ptr, sub.child_idx, sub.n_nodes)
    ot.forward(sub.child_ptr, sub.child_idx, x, w.W, w.U, w.b)


def time_oracle(w: wl.Workload, budget_s: float):
    """nodes/s of the checker on a bounded sample of whole trees (one thread)."""
    try:
        from threadpoolctl import threadpool_limits
        ctx = threadpool_limits(limits=1)
    except Exception:  # pragma: no cover
        import contextlib
        ctx = contextlib.nullcontext()
    with ctx:
        n = 2
        while True:
            sub, x = oracle_sample(w, n)
            t0 = time.perf_counter()
            oracle_step(w, sub, x)
            dt = time.perf_counter() - t0
            if dt * 2.2 > budget_s or n >= w.forest.n_trees:
                break
            n = min(w.forest.n_trees, max(n + 1, int(n * min(8.0, 0.8 * budget_s / max(dt, 1e-4)))))
        # a workload the checker finishes quickly is repeated until the sample is worth the budget
        runs = max(1, int(0.8 * budget_s / max(dt, 1e-4)))
        if runs > 1:
            t0 = time.perf_counter()
            for _ in range(runs):
                oracle_step(w, sub, x)
            dt = (time.perf_counter() - t0) / runs
    return (sub.n_nodes / dt,
            f"first {sub.n_trees} of {w.forest.n_trees} trees ({sub.n_nodes} nodes), {runs} run(s), {dt:.2f} s each",
            sub.n_trees)


def _oracle_worker(task):
    """One process of the parallel baseline: the checker, as it stands, over its share of the trees (one thread)."""
    child_ptr, child_idx, x, W, U, b, n_nodes = task
    from threadpoolctl import threadpool_limits
    from oracle import schedule as osched
    from oracle import treelstm as ot
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        osched.schedule(child_ptr, child_idx, n_nodes)
        ot.forward(child_ptr, child_idx, x, W, U, b)
        return n_nodes, time.perf_counter() - t0


def time_oracle_parallel(w: wl.Workload, trees_per_worker: int, max_workers: int = 32):
    """nodes/s of the checker with the trees dealt out over worker processes (trees are independent units).
    Workers are started with `spawn`: the parent process already holds a CUDA context."""
    import multiprocessing as mp
    try:
        avail = len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        avail = os.cpu_count() or 1
    cores = max(1, min(avail, max_workers, w.forest.n_trees // max(trees_per_worker, 1) or 1))
    tasks = []
    for k in range(cores):
        trees = np.arange(k * trees_per_worker, min((k + 1) * trees_per_worker, w.forest.n_trees))
        sub, nodes = wl.subforest(w.forest, trees)
        tasks.append((sub.child_ptr, sub.child_idx, w.x_rows(nodes), w.W, w.U, w.b, sub.n_nodes))
    one, one_nodes = wl.subforest(w.forest, np.arange(1))
    warm = (one.child_ptr, one.child_idx, w.x_rows(one_nodes), w.W, w.U, w.b, one.n_nodes)
    ctx = mp.get_context("spawn")
    with ctx.Pool(cores) as pool:
        pool.map(_oracle_worker, [warm] * cores, chunksize=1)  # untimed: process start-up and imports
        t0 = time.perf_counter()
        done = pool.map(_oracle_worker, tasks, chunksize=1)
        dt = time.perf_counter() - t0
    nodes = sum(d[0] for d in done)
    return nodes / dt, cores, f"{cores} processes x {trees_per_worker} trees ({nodes} nodes), {dt:.2f} s"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.make_workload(args.config)
    from threadpoolctl import threadpool_limits
    with threadpool_limits(limits=1):
        n_trees = 2
        sub, x = oracle_sample(w, n_trees)
        t0 = time.perf_counter()
        oracle_step(w, sub, x)
        per_node = (time.perf_counter() - t0) / sub.n_nodes
        # size the per-step sample so that the whole run stays within about two minutes
        total_steps = args.steps + args.warmup
        target_nodes = max(sub.n_nodes, int(90.0 / max(total_steps, 1) / per_node))
        mean_tree = w.forest.n_nodes / w.forest.n_trees
        n_trees = int(max(1, min(w.forest.n_trees, target_nodes / mean_tree)))
        sub, x = oracle_sample(w, n_trees)
        for _ in range(args.warmup):
            oracle_step(w, sub, x)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            oracle_step(w, sub, x)
        dt = time.perf_counter() - t0
    value = sub.n_nodes * args.steps / dt
    sample = f"first {sub.n_trees} of {w.forest.n_trees} trees ({sub.n_nodes} nodes) per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"config {args.config} ({w.name})", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def algorithmic_work(w: wl.Workload, n_leaves: int):
    """Minimal flops and bytes of one forward (what the method must compute and touch): every row once, the weights
    once at their own type, nothing round-tripped."""
    f = w.forest
    N, E, D, H = f.n_nodes, f.n_edges, w.D, w.H
    n_int = N - n_leaves
    flops = n_leaves * 6 * D * H + n_int * 8 * D * H + n_int * 6 * H * H + E * 2 * H * H
    sx = 2 if w.precision == "bf16" else 4
    ws = 2 if w.precision == "bf16" else 4
    bytes_ = N * D * sx + N * 2 * 4 * H + E * 2 * 4 * H + 4 * (2 * N + E) * 3 + (D + H) * 4 * H * ws
    return flops, bytes_


def level_loop_bytes(w: wl.Workload, n_leaves: int):
    """(algorithmic, design) bytes of the level loop alone.  Algorithmic: h and c rows of the internal nodes out, h and c
    rows of every child in, the recurrent weights once at their own type, the index arrays.  Design: what the kernels
    add on top of that by construction (the fp32 input-projection rows of the internal nodes they read back; the
    bf16 copies of h the tensor-core paths keep)."""
    f = w.forest
    n_int = f.n_nodes - n_leaves
    H = w.H
    ws = 2 if w.precision == "bf16" else 4
    algorithmic = n_int * 2 * H * 4 + f.n_edges * 2 * H * 4 + 4 * H * H * ws + 4 * (2 * n_int + f.n_edges)
    design = n_int * 4 * H * 4
    if w.precision == "bf16":
        design += (n_int + f.n_edges) * H * 2
    return algorithmic, design


# ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch (of all launches of one step, for the per-level loop)
# of the named kernels on the named workload, from the captures summarised under profiles/; None where a kernel has
# changed since its counters were taken.
MEASURED_TRAFFIC = {
    ("small_levels_f32_kernel", 1): 2231040,            # whole workload captured, one launch
    ("small_levels_kernel", 2): 5665792,                # whole workload captured, one launch
    ("small_levels_kernel", 4): 896706560,              # whole workload captured, one launch
    # per-level loop = all childsum_kernel, gemm_tc_kernel<EPI_F> and gemm_tc_kernel<EPI_LEVEL> launches of one step
    ("per-level loop", 3): 1656050000,                  # whole workload captured (12 levels, 36 launches)
    # captured on 8192 of the 65536 trees (194583 nodes: 2775 MB) and scaled by the node count: every row is read and
    # written a fixed number of times, so traffic grows in proportion
    ("per-level loop", 5): int(2775.2e6 * (1571637 / 194583)),
    # input projection of workload 5 (CTA pairs, eight epilogue warps): one launch captured on the same 8192 trees
    # (409.06 MB read, 2035.62 MB written), scaled
    ("gemm_tc2_kernel<EPI_XPROJ8>", 5): int(2444.68e6 * (1571637 / 194583)),
}


def roofline_of(job, phases, t_step_s, pk):
    """Roofline object of the dominant kernel of one step, the same for both phases, and the whole step against its
    binding bound.

    phases: per step (input projection ms, level loop ms, batching analysis ms) from CUDA events recorded by the
    library on the launching stream around those kernels.  The tensor peak is the burst figure of the measured
    bf16 GEMM (the higher of the two measured ones) for every workload.
    """
    w = job.w
    f = w.forest
    N, E, D, H = f.n_nodes, f.n_edges, w.D, w.H
    n_int = N - job.n_leaves
    xproj_ms = statistics.mean(p[0] for p in phases)
    lvl_ms = statistics.mean(p[1] for p in phases)
    flops, bytes_ = algorithmic_work(w, job.n_leaves)
    tensor_peak = pk["bf16_tflops"]
    t_tensor = flops / (tensor_peak * 1e12) if w.precision == "bf16" else 0.0
    t_hbm = bytes_ / (pk["hbm_gbs"] * 1e9)
    path_frac = max(t_tensor, t_hbm) / t_step_s

    # input projection: algorithmic flops = three gate blocks for leaves, four for internal nodes
    xflops = (job.n_leaves * 6 + n_int * 8) * D * H
    x_ach = xflops / (xproj_ms * 1e-3) / 1e12 if xproj_ms > 0 else 0.0
    lbytes, ldesign = level_loop_bytes(w, job.n_leaves)
    l_ach = lbytes / (lvl_ms * 1e-3) / 1e9 if lvl_ms > 0 else 0.0
    lflops = n_int * 6 * H * H + E * 2 * H * H
    if w.precision != "bf16":
        lkernel = "small_levels_f32_kernel" if w.H <= 192 else "persistent_kernel / level_kernel (fp32 ALUs)"
    elif job.small:
        lkernel = "small_levels_kernel"
    else:
        lkernel = "per-level loop"
    phases_out = {
        "input_projection": {"kernel": "tcgen05 GEMM (gemm_tc_kernel / gemm_tc2_kernel)" if w.precision == "bf16" else "xproj_simt_kernel",
                             "ms": xproj_ms, "flops": xflops, "tflops": x_ach,
                             "frac_of_tensor_peak": x_ach / tensor_peak if w.precision == "bf16" else None},
        "level_loop": {"kernel": lkernel, "ms": lvl_ms, "algorithmic_bytes": lbytes, "design_bytes": ldesign,
                       "gbs": l_ach, "frac_of_hbm_peak": l_ach / pk["hbm_gbs"], "flops": lflops,
                       "tflops": lflops / (lvl_ms * 1e-3) / 1e12 if lvl_ms > 0 else 0.0},
        "schedule_ms": statistics.mean(p[2] for p in phases),
    }
    if w.precision == "bf16" and xproj_ms >= lvl_ms:
        # the library's own choice: CTA pairs with eight epilogue warps from 128 tiles per pair on (148 SMs)
        Hp = (H + 63) // 64 * 64
        many = not job.small and ((N + 255) // 256) * (4 * Hp // 256) >= 128 * 74
        kernel = "gemm_tc2_kernel<EPI_XPROJ8>" if many else "gemm_tc_kernel<EPI_XPROJ>"
        roof = {"bound": "tensor", "kernel": kernel, "achieved": x_ach, "peak": tensor_peak, "unit": "TFLOP/s",
                "frac": x_ach / tensor_peak, "frac_of_sustained_peak": x_ach / pk["bf16_tflops_sustained"]}
    else:
        kernel = lkernel
        roof = {"bound": "hbm", "kernel": kernel, "achieved": l_ach, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": l_ach / pk["hbm_gbs"], "algorithmic_bytes": lbytes, "design_bytes": ldesign}
        if kernel == "per-level loop":
            roof["kernel"] = "per-level loop: childsum_kernel + gemm_tc_kernel<EPI_F> + gemm_tc_kernel<EPI_LEVEL> per level"
    roof["traffic"] = MEASURED_TRAFFIC.get((kernel, w.index))
    roof["peak_source"] = pk["source"]
    roof["ms_per_launch"] = xproj_ms if roof["bound"] == "tensor" else lvl_ms
    roof["xproj_ms"] = xproj_ms
    roof["levels_ms"] = lvl_ms
    roof["schedule_ms"] = phases_out["schedule_ms"]   # batching analysis alone (start of step to start of forward)
    return roof, path_frac, phases_out


class GpuJob:
    """Device-resident inputs and buffers of one workload, and the calls of one step."""

    def __init__(self, w: wl.Workload, device, mode):
        import torch
        from paper_1904_07421_b200 import jdb
        self.torch, self.jdb, self.w, self.mode = torch, jdb, w, mode
        f = w.forest
        self.forest = jdb.forest_to_device(f.child_ptr, f.child_idx, device)
        self.precision = jdb.BF16 if w.precision == "bf16" else jdb.FP32
        dt = torch.bfloat16 if self.precision == jdb.BF16 else torch.float32
        table = torch.from_numpy(w.table).to(device).to(dt)
        token = torch.from_numpy(w.token.astype(np.int64)).to(device)
        self.ldx = (w.D + 7) // 8 * 8
        self.x = torch.zeros((f.n_nodes, self.ldx), dtype=dt, device=device)
        self.x[:, :w.D] = table[token]
        del table, token
        self.packed = jdb.jdb_pack_weights(*(torch.from_numpy(a).to(device) for a in (w.W, w.U, w.b)), self.precision)
        self.sched = jdb.alloc_schedule(f.n_nodes, device)
        self.sws = jdb.schedule_workspace(self.forest)
        self.ldh = (w.H + 3) // 4 * 4
        self.h = torch.empty((f.n_nodes, self.ldh), dtype=torch.float32, device=device)
        self.c = torch.empty((f.n_nodes, self.ldh), dtype=torch.float32, device=device)
        jdb.jdb_schedule(self.forest, self.sched, self.sws)
        self.n_levels, self.n_leaves = self.sched.n_levels, self.sched.n_leaves
        self.level_sizes = np.diff(self.sched.level_ptr[:self.n_levels + 1].cpu().numpy()).tolist()
        self.small = self.precision == jdb.BF16 and w.H <= 192 and mode != jdb.MODE_PER_LEVEL
        # the cooperative level loops read the level count on the device, so the analysis need not synchronise
        # and the forward can defer its status to one check after the timed loop; per-level launches need the
        # counts on the host, so there the analysis synchronises inside the step
        self.async_schedule = self.small or self.precision == jdb.FP32
        if self.async_schedule:
            self.sched.n_leaves = -1  # size the workspace for a schedule whose counts stay on the device
        self.fws = jdb.forward_workspace(self.forest, self.sched, w.D, w.H, self.precision)
        self.events = None
        self.plan = jdb.StepPlan(self.forest, self.sched, self.sws, self.x, self.packed, w.D, w.H, self.precision,
                                 self.h, self.c, self.fws, mode=mode, async_schedule=self.async_schedule)

    def step(self):
        self.plan.set_events(self.events)
        self.plan.run()

    def launches_per_step(self):
        """Kernels of this library launched by one step (memsets and copies not counted)."""
        jdb = self.jdb
        sched = 1 if self.forest.n_nodes <= 6144 else 4 + 3 * 2
        levels = max(self.n_levels - 1, 0)
        if self.precision == jdb.FP32:
            persistent = self.mode == jdb.MODE_PERSISTENT or (self.mode == jdb.MODE_AUTO and (self.w.H <= 192 or self.n_levels > 6))
            return sched + 1 + (1 if persistent else levels)
        if self.small:
            return sched + 2 + (1 if levels else 0)   # level-order copy, projection GEMM, cooperative level loop
        return sched + 2 + 3 + 3 * levels             # + three layout kernels, and child sums + two GEMMs per level


def time_steps(job: GpuJob, steps: int, warmup: int, flush, timed_events=False):
    """Per-step CUDA-event times (ms) on the current stream, L2 flushed between steps."""
    torch = job.torch
    for _ in range(warmup):
        job.step()
    torch.cuda.synchronize()
    total, level_ms = [], []
    for _ in range(steps):
        flush.add_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if timed_events:
            job.events = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e0.record()
        job.step()
        e1.record()
        e1.synchronize()
        total.append(e0.elapsed_time(e1))
        if timed_events:
            level_ms.append((job.events[0].elapsed_time(job.events[1]), job.events[1].elapsed_time(job.events[2]),
                             e0.elapsed_time(job.events[0])))
    job.events = None
    job.plan.status()  # raises if any step recorded a malformed forest or a timed-out wait
    return total, level_ms


def time_e2e(w: wl.Workload, job: GpuJob, steps: int, warmup: int, flush, device, roots_only: bool = False):
    """The same step through the host-buffer entry point: pinned host arrays in, pinned host arrays out, the
    copies inside the timed region.  Returns (per-step ms, h2d bytes, d2h bytes)."""
    torch, jdb = job.torch, job.jdb
    f = w.forest
    dt = torch.bfloat16 if job.precision == jdb.BF16 else torch.float32
    hx = torch.from_numpy(w.x_full()).to(dt).pin_memory()
    hcp, hci = torch.from_numpy(f.child_ptr).pin_memory(), torch.from_numpy(f.child_idx).pin_memory()
    rows = f.n_nodes - f.n_edges if roots_only else f.n_nodes   # with JDB_FLAG_ROOTS_ONLY only the roots' states come back
    flags = jdb.FLAG_ROOTS_ONLY if roots_only else 0
    hh = torch.empty((rows, w.H), dtype=torch.float32).pin_memory()
    hc = torch.empty((rows, w.H), dtype=torch.float32).pin_memory()
    x_dtype = jdb.BF16 if dt == torch.bfloat16 else jdb.FP32
    hws = jdb.forward_host_workspace(f.n_nodes, f.n_edges, w.D, w.H, job.precision, x_dtype, device)
    for _ in range(max(warmup, 3)):
        jdb.jdb_treelstm_forward_host(hcp, hci, hx, job.packed, w.D, w.H, job.precision, hh, hc, hws, flags=flags)
    torch.cuda.synchronize()
    ms = []
    for _ in range(steps):
        flush.add_(1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        jdb.jdb_treelstm_forward_host(hcp, hci, hx, job.packed, w.D, w.H, job.precision, hh, hc, hws, flags=flags)
        e1.record()
        e1.synchronize()
        ms.append(e0.elapsed_time(e1))
    h2d = hcp.numel() * 4 + hci.numel() * 4 + hx.numel() * hx.element_size()
    d2h = hh.numel() * 4 + hc.numel() * 4
    return ms, h2d, d2h


def time_e2e_pipelined(w: wl.Workload, job_precision, packed, steps: int, warmup: int, flush, device, chunks: int = 8, slots: int = 3):
    """The same end-to-end step with the forest handed over in `chunks` groups of whole trees through jdb_online_*: the
    copies in of one group, the execution of another and the copies back of a third overlap.  Returns per-step ms."""
    import torch
    from paper_1904_07421_b200 import jdb
    f = w.forest
    dt = torch.bfloat16 if job_precision == jdb.BF16 else torch.float32
    bounds = np.linspace(0, f.n_trees, min(chunks, f.n_trees) + 1).astype(np.int64)
    parts = []
    for a, b in zip(bounds[:-1], bounds[1:]):
        sub, nodes = wl.subforest(f, np.arange(a, b))
        parts.append((torch.from_numpy(sub.child_ptr.astype(np.int32)).pin_memory(), torch.from_numpy(sub.child_idx.astype(np.int32)).pin_memory(),
                      torch.from_numpy(w.x_rows(nodes)).to(dt).pin_memory(),
                      torch.empty((len(nodes), w.H), dtype=torch.float32).pin_memory(),
                      torch.empty((len(nodes), w.H), dtype=torch.float32).pin_memory(), sub.n_edges))
    on = jdb.Online(slots, max(p[3].shape[0] for p in parts), max(p[5] for p in parts), packed, w.D, w.H, job_precision,
                    jdb.BF16 if dt == torch.bfloat16 else jdb.FP32, device)

    def step():
        tickets = [on.submit(*p[:5]) for p in parts]
        for t in tickets:
            on.wait(t)

    for _ in range(max(warmup, 3)):
        step()
    torch.cuda.synchronize()
    ms = []
    for _ in range(steps):
        flush.add_(1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        step()
        torch.cuda.synchronize()
        e1.record()
        e1.synchronize()
        ms.append(e0.elapsed_time(e1))
    on.close()
    return ms


def time_head(w: wl.Workload, job: GpuJob, flush, pk, Hs: int = 50, K: int = 5, reps: int = 10):
    """The relatedness head over the forest's root states (pairs of consecutive trees): time per call and the
    fraction of the copy bandwidth its algorithmic bytes (two root rows per pair) reach.  Not part of `value`."""
    torch, jdb = job.torch, job.jdb
    rng = np.random.default_rng(7)
    H = w.H
    dev = job.h.device
    mk = lambda *shape: torch.from_numpy(rng.uniform(-0.3, 0.3, shape).astype(np.float32)).to(dev)
    Wx, Wp, bh, Wq, bq = mk(Hs, H), mk(Hs, H), mk(Hs), mk(K, Hs), mk(K)
    roots = torch.from_numpy(w.forest.roots.astype(np.int32)).to(dev)
    left, right = roots[0::2].contiguous(), roots[1::2].contiguous()
    n_pairs = int(min(left.numel(), right.numel()))
    left, right = left[:n_pairs], right[:n_pairs]
    if n_pairs == 0:
        return None
    ms = []
    for _ in range(reps + 3):
        flush.add_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        jdb.jdb_relatedness_head(job.h, left, right, Wx, Wp, bh, Wq, bq, want_p=False)
        e1.record()
        e1.synchronize()
        ms.append(e0.elapsed_time(e1))
    t = statistics.median(ms[3:])
    bytes_ = n_pairs * 2 * H * 4
    return {"pairs": n_pairs, "ms": t, "pairs_per_s": n_pairs / (t * 1e-3), "algorithmic_bytes": bytes_,
            "frac_of_hbm_peak": bytes_ / (t * 1e-3) / 1e9 / pk["hbm_gbs"], "head_hidden": Hs, "classes": K}


def time_training(idx: int, w: wl.Workload, device, flush, steps: int = 5, warmup: int = 3):
    """One training pass in fp32 (Section 5 reports training beside inference): batching analysis, forward, and the
    backward pass over the same depth table with the loss on the root states.  Not part of `value`."""
    import torch
    from paper_1904_07421_b200 import jdb
    f = w.forest
    D, H = w.D, w.H
    forest = jdb.forest_to_device(f.child_ptr, f.child_idx, device)
    x = torch.from_numpy(w.x_full()).to(device)
    W, U, b = (torch.from_numpy(a).to(device) for a in (w.W, w.U, w.b))
    packed = jdb.jdb_pack_weights(W, U, b, jdb.FP32)
    sched = jdb.alloc_schedule(f.n_nodes, device)
    sws = jdb.schedule_workspace(forest)
    jdb.jdb_schedule(forest, sched, sws)
    n_int = f.n_nodes - sched.n_leaves
    fws = jdb.forward_workspace(forest, sched, D, H, jdb.FP32)
    bws = torch.empty(jdb.lib().jdb_treelstm_backward_workspace_bytes(f.n_nodes, f.n_edges, n_int, H), dtype=torch.uint8, device=device)
    h = torch.empty((f.n_nodes, H), dtype=torch.float32, device=device)
    c = torch.empty_like(h)
    gh = torch.zeros_like(h)
    rng = np.random.default_rng(11)
    roots = torch.from_numpy(f.roots.astype(np.int64)).to(device)
    gh[roots] = torch.from_numpy(rng.standard_normal((f.n_trees, H)).astype(np.float32)).to(device)
    fwd, bwd = [], []
    for it in range(warmup + steps):
        flush.add_(1)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        jdb.jdb_schedule(forest, sched, sws)
        jdb.jdb_treelstm_forward(forest, sched, x, packed, D, H, jdb.FP32, h=h, c=c, ws=fws)
        e[1].record()
        jdb.jdb_treelstm_backward(forest, sched, x, W, U, b, h, c, gh, None, ws=bws)
        e[2].record()
        e[2].synchronize()
        if it >= warmup:
            fwd.append(e[0].elapsed_time(e[1]))
            bwd.append(e[1].elapsed_time(e[2]))
    tf, tb = statistics.median(fwd), statistics.median(bwd)
    # mixed precision: the tensor-core forward (bf16 operands) feeding the same fp32 backward pass
    tf16 = None
    if w.precision == "bf16":
        packed16 = jdb.jdb_pack_weights(W, U, b, jdb.BF16)
        x16 = x.to(torch.bfloat16)
        fws16 = jdb.forward_workspace(forest, sched, D, H, jdb.BF16)
        f16 = []
        for it in range(warmup + steps):
            flush.add_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            jdb.jdb_schedule(forest, sched, sws)
            jdb.jdb_treelstm_forward(forest, sched, x16, packed16, D, H, jdb.BF16, h=h, c=c, ws=fws16)
            e1.record()
            e1.synchronize()
            if it >= warmup:
                f16.append(e0.elapsed_time(e1))
        tf16 = statistics.median(f16)
        del packed16, x16, fws16
    flops_b = 3.0 * (8.0 * f.n_nodes * D * H + 6.0 * n_int * H * H + 2.0 * f.n_edges * H * H)
    return {"config": idx, "workload": w.name, "nodes": f.n_nodes, "trees": f.n_trees, "D": D, "H": H, "dtype": "f32",
            "step": "jdb_schedule + jdb_treelstm_forward + jdb_treelstm_backward (loss on the roots)",
            "forward_ms": tf, "backward_ms": tb, "nodes_per_s": f.n_nodes / ((tf + tb) * 1e-3),
            "trees_per_s": f.n_trees / ((tf + tb) * 1e-3),
            "forward_bf16_ms": tf16, "trees_per_s_bf16_forward": (f.n_trees / ((tf16 + tb) * 1e-3)) if tf16 else None,
            "backward_flops": flops_b,
            "backward_tflops": flops_b / (tb * 1e-3) / 1e12,
            "backward_frac_of_fp32_alu_peak": flops_b / (tb * 1e-3) / 1e12 / FP32_ALU_PEAK_TFLOPS,
            "launches_backward": 4 + 2 + 3 + 3 * max(sched.n_levels - 1, 0) + 1 + 5}


def time_batcher(idx: int, w: wl.Workload, device, flush, steps: int = 5, warmup: int = 3):
    """Section 4.2's table for nodes of two kinds (a Child-Sum and an N-ary cell drawn per node) and its execution slot
    by slot in fp32: jdb_batch_plan + jdb_cells_forward on the workload's forest.  Not part of `value`."""
    import torch
    from paper_1904_07421_b200 import jdb
    f = w.forest
    D, H = w.D, w.H
    rng = np.random.default_rng(13)
    kids = np.diff(f.child_ptr)
    arity = int(max(1, kids.max()))
    if arity > 8:
        return None
    key_h = rng.integers(0, 2, size=f.n_nodes).astype(np.int32)
    forest = jdb.forest_to_device(f.child_ptr, f.child_idx, device)
    x = torch.from_numpy(w.x_full()).to(device)
    Un = (rng.standard_normal(((3 + arity) * H, arity * H)) / np.sqrt(arity * H)).astype(np.float32)
    cells = [(jdb.CELL_CHILDSUM, 0, *(torch.from_numpy(a).to(device) for a in (w.W, w.U, w.b))),
             (jdb.CELL_NARY, arity, *(torch.from_numpy(a).to(device) for a in (w.W, Un, w.b)))]
    key = torch.from_numpy(key_h).to(device)
    sched = jdb.jdb_schedule(forest)
    h = torch.empty((f.n_nodes, H), dtype=torch.float32, device=device)
    c = torch.empty_like(h)
    ws = torch.empty(jdb.lib().jdb_cells_forward_workspace_bytes(f.n_nodes, f.n_edges, H, arity, 2), dtype=torch.uint8, device=device)
    t_plan, t_run = [], []
    plan = None
    for it in range(warmup + steps):
        flush.add_(1)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        plan = jdb.jdb_batch_plan(forest, sched, key, 2)
        e[1].record()
        jdb.jdb_cells_forward(forest, plan, key, cells, x, D, H, h=h, c=c, ws=ws)
        e[2].record()
        e[2].synchronize()
        if it >= warmup:
            t_plan.append(e[0].elapsed_time(e[1]))
            t_run.append(e[1].elapsed_time(e[2]))
    tp, tr = statistics.median(t_plan), statistics.median(t_run)
    internal = kids > 0
    flops = (8.0 * f.n_nodes * D * H
             + float(np.sum((6.0 + 2.0 * kids) * H * H * (internal & (key_h == 0))))
             + float(np.sum(2.0 * (3 + arity) * kids * H * H * (internal & (key_h == 1)))))
    return {"config": idx, "workload": w.name, "nodes": f.n_nodes, "levels": int(sched.n_levels), "slots": int(plan.n_slots),
            "cells": ["childsum", f"nary(arity {arity})"], "D": D, "H": H, "dtype": "f32",
            "step": "jdb_batch_plan + jdb_cells_forward", "plan_ms": tp, "forward_ms": tr,
            "nodes_per_s": f.n_nodes / ((tp + tr) * 1e-3), "flops": flops, "tflops": flops / (tr * 1e-3) / 1e12,
            "frac_of_fp32_alu_peak": flops / (tr * 1e-3) / 1e12 / FP32_ALU_PEAK_TFLOPS}


def time_online(device, slots: int = 4, n_requests: int = 64, index: int = 2):
    """A stream of requests (forests of workload 2's shape with 16 to 256 trees, pinned host buffers) through the
    one-call host entry one after the other, and through jdb_online_* with `slots` requests in flight.  Host clock
    around the whole stream, device idle on both sides.  Not part of `value`."""
    import time
    import torch
    from paper_1904_07421_b200 import jdb
    rng = np.random.default_rng(17)
    base = wl.make_workload(index, n_trees=4)
    precision = jdb.BF16 if base.precision == "bf16" else jdb.FP32
    dt = torch.bfloat16 if precision == jdb.BF16 else torch.float32
    packed = jdb.jdb_pack_weights(*(torch.from_numpy(a).to(device) for a in (base.W, base.U, base.b)), precision)
    reqs = []
    for k in range(n_requests):
        wk = wl.make_workload(index, n_trees=int(rng.integers(16, 257)), seed=1000 + k)
        f = wk.forest
        x = torch.from_numpy(base.table[wk.token % base.table.shape[0]]).to(dt).pin_memory()
        reqs.append((torch.from_numpy(f.child_ptr.astype(np.int32)).pin_memory(), torch.from_numpy(f.child_idx.astype(np.int32)).pin_memory(), x,
                     torch.empty((f.n_nodes, wk.H), dtype=torch.float32).pin_memory(),
                     torch.empty((f.n_nodes, wk.H), dtype=torch.float32).pin_memory(), f.n_nodes, f.n_trees, f.n_edges))
    max_n, max_e = max(r[5] for r in reqs), max(r[7] for r in reqs)
    ws = jdb.forward_host_workspace(max_n, max_e, base.D, base.H, precision, precision, device)
    on = jdb.Online(slots, max_n, max_e, packed, base.D, base.H, precision, precision, device)

    def serial():
        for r in reqs:
            jdb.jdb_treelstm_forward_host(r[0], r[1], r[2], packed, base.D, base.H, precision, r[3], r[4], ws)

    def online():
        tickets = [on.submit(*r[:5]) for r in reqs]
        for t in tickets:
            on.wait(t)

    out = {}
    for name, fn_ in (("one_call_entries", serial), ("online", online)):
        fn_()
        torch.cuda.synchronize()
        ts = []
        for _ in range(5):
            t0 = time.perf_counter()
            fn_()
            torch.cuda.synchronize()
            ts.append(time.perf_counter() - t0)
        out[name] = statistics.median(ts)
    on.close()
    nodes, trees = sum(r[5] for r in reqs), sum(r[6] for r in reqs)
    return {"workload": f"{n_requests} requests of workload {index}'s shape, 16-256 trees each ({trees} trees, {nodes} nodes), "
                        "pinned host buffers in and out", "slots": slots,
            "one_call_entries": {"seconds": out["one_call_entries"], "requests_per_s": n_requests / out["one_call_entries"],
                                 "nodes_per_s": nodes / out["one_call_entries"]},
            "online": {"seconds": out["online"], "requests_per_s": n_requests / out["online"], "nodes_per_s": nodes / out["online"]},
            "speedup": out["one_call_entries"] / out["online"]}


def rank_workload(config: int, rank: int, n_trees=None) -> wl.Workload:
    """Every rank draws its own forest of the workload's shape (weak scaling over independent trees)."""
    return wl.make_workload(config, n_trees=n_trees, seed=None if rank == 0 else wl.BASE_SEED + config + 1000 * rank)


def job_totals(seconds: float, nodes: int, world: int, device):
    """Whole-job figures: the slowest rank's time and the nodes all ranks processed (no data-path collective)."""
    if world == 1:
        return seconds, float(nodes)
    import torch
    import torch.distributed as dist
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    n = torch.tensor([float(nodes)], dtype=torch.float64, device=device)
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


def config_entry(idx, w, job, times, steps, value, roofline, path_frac, phases):
    f = w.forest
    return {"config": idx, "workload": w.name, "nodes": f.n_nodes, "edges": f.n_edges, "levels": job.n_levels,
            "level_sizes": job.level_sizes, "batching_ratio": f.n_nodes / max(job.n_levels, 1), "steps": steps,
            "ms_per_step": sum(times) / len(times), "ms_median": statistics.median(times), "ms_min": min(times),
            "value": value, "roofline": roofline, "path_frac_of_roofline": path_frac, "phases": phases}


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_1904_07421_b200 import jdb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.rendezvous_only:
        # a check of the launcher that needs no GPU: the ranks meet over gloo, reduce the totals, rank 0 prints
        dist.init_process_group("gloo")
        w = rank_workload(1, rank)
        t_s, total_nodes = job_totals(1.0 + rank, w.forest.n_nodes, world, torch.device("cpu"))
        if rank == 0:
            print(json.dumps({"metric": METRIC, "n_gpus": world, "rendezvous_only": True, "max_seconds": t_s,
                              "total_nodes": total_nodes}))
        dist.barrier()
        dist.destroy_process_group()
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    if local_rank >= torch.cuda.device_count():
        raise SystemExit(f"rank {rank} has no GPU: {torch.cuda.device_count()} visible, {world} ranks")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    jdb.lib()

    if args.training_only:
        flush = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=device)
        wt = wl.make_workload(args.training_only, n_trees=args.trees)
        print(json.dumps({"training": [time_training(args.training_only, wt, device, flush, args.steps, args.warmup)],
                          "keyed_batcher": [time_batcher(args.training_only, wt, device, flush, args.steps, args.warmup)],
                          "online_requests": time_online(device) if args.training_only == 2 else None}))
        return
    pk = peaks()
    mode = {"auto": jdb.MODE_AUTO, "level": jdb.MODE_PER_LEVEL, "persistent": jdb.MODE_PERSISTENT}[args.mode]
    w = rank_workload(args.config, rank, args.trees)
    f = w.forest
    job = GpuJob(w, device, mode)
    flush = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=device)

    sampler = ClockSampler(local_rank)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    for _ in range(args.warmup):
        job.step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler.start()
    times, phases = time_steps(job, args.steps, 0, flush, timed_events=True)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    t_s, total_nodes = job_totals(sum(times) / 1e3, f.n_nodes, world, device)
    value = total_nodes * args.steps / t_s
    roofline, path_frac, phases_out = roofline_of(job, phases, t_s / args.steps, pk)
    main_entry = config_entry(args.config, w, job, times, args.steps, value, roofline, path_frac, phases_out)
    n_levels_main, launches_main = job.n_levels, job.launches_per_step()
    precision_main, packed_main = job.precision, job.packed

    # the workload's scoring step (Section 5: relatedness of sentence pairs): consecutive trees form a pair
    head = time_head(w, job, flush, pk)

    # end to end from pinned host buffers through the host entry point (the resident buffers are released first)
    job.plan = None
    job.x = job.h = job.c = job.fws = job.sws = None
    torch.cuda.empty_cache()
    e2e_ms, h2d, d2h = time_e2e(w, job, args.steps, args.warmup, flush, device)
    t_e2e_s, _ = job_totals(sum(e2e_ms) / 1e3, f.n_nodes, world, device)
    e2e_value = total_nodes * args.steps / t_e2e_s
    torch.cuda.empty_cache()
    roots_ms, _, roots_d2h = time_e2e(w, job, args.steps, args.warmup, flush, device, roots_only=True)
    t_roots_s, _ = job_totals(sum(roots_ms) / 1e3, f.n_nodes, world, device)
    torch.cuda.empty_cache()
    pipe_ms = time_e2e_pipelined(w, precision_main, packed_main, args.steps, args.warmup, flush, device)
    t_pipe_s, _ = job_totals(sum(pipe_ms) / 1e3, f.n_nodes, world, device)
    pipe_value = total_nodes * args.steps / t_pipe_s
    del job
    torch.cuda.empty_cache()

    if rank == 0:
        per_config = []
        if args.all_configs and world == 1:
            for idx in (1, 2, 3, 4, 5):
                if idx == args.config:
                    per_config.append(main_entry)
                    continue
                wi = wl.make_workload(idx)
                ji = GpuJob(wi, device, mode)
                ti, ph = time_steps(ji, args.steps, args.warmup, flush, timed_events=True)
                ri, pf, po = roofline_of(ji, ph, sum(ti) / 1e3 / args.steps, pk)
                per_config.append(config_entry(idx, wi, ji, ti, args.steps, wi.forest.n_nodes * args.steps / (sum(ti) / 1e3), ri, pf, po))
                del ji, wi
                torch.cuda.empty_cache()
        training, batcher = [], []
        if args.all_configs and world == 1:
            for idx in (1, 2, 3, 4):
                training.append(time_training(idx, wl.make_workload(idx), device, flush))
                torch.cuda.empty_cache()
            for idx in (1, 2, 3):
                b = time_batcher(idx, wl.make_workload(idx), device, flush)
                if b is not None:
                    batcher.append(b)
                torch.cuda.empty_cache()
        online = time_online(device) if (args.all_configs and world == 1) else None
        cpu_v, cpu_sample, cpu_trees = time_oracle(w, args.cpu_budget)
        cpu_par = None
        if args.cpu_budget >= 1.0:
            pv, pcores, psample = time_oracle_parallel(w, max(1, cpu_trees))
            cpu_par = {"value": pv, "unit": UNIT, "cores": pcores, "kind": "oracle", "sample": psample}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * t_s / args.steps, "ms_median": statistics.median(times), "ms_min": min(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if w.precision == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": f"config {args.config} ({w.name}): {f.n_trees} trees, {f.n_nodes} nodes, "
                                   f"{f.n_edges} edges, {n_levels_main} levels, D={w.D}, H={w.H}",
                       "step": "jdb_schedule + jdb_treelstm_forward", "mode": args.mode,
                       **({"reduced_to_trees": args.trees} if args.trees else {}),
                       "l2": "256 MiB buffer rewritten between timed steps", "parallelism": f"tree-sharded x{world}"},
            "clocks": clocks,
            # the better of the two ways a caller has: one call for the whole forest, or the forest handed over in eight
            # groups of whole trees through jdb_online_* (three slots), whose copies and execution overlap
            "e2e": {"value": max(e2e_value, pipe_value), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": 1e3 * min(t_e2e_s, t_pipe_s) / args.steps,
                    "entry": "jdb_online_* (8 groups of trees, 3 slots)" if pipe_value > e2e_value else "jdb_treelstm_forward_host",
                    "one_call": {"value": e2e_value, "ms_per_step": 1e3 * t_e2e_s / args.steps},
                    "pipelined": {"value": pipe_value, "ms_per_step": 1e3 * t_pipe_s / args.steps},
                    # the one call with JDB_FLAG_ROOTS_ONLY: only the roots' states cross back (what a sentence-level
                    # task reads); not the line's e2e value, which returns every node's state
                    "roots_only": {"value": total_nodes * args.steps / t_roots_s, "ms_per_step": 1e3 * t_roots_s / args.steps,
                                   "d2h_bytes_per_step": roots_d2h}},
            "gpu_launches": launches_main * args.steps,
            "roofline": roofline,
            "path_frac_of_roofline": path_frac,
            "phases": phases_out,
            "relatedness_head": head,
            "training": training,
            "keyed_batcher": batcher,
            "online_requests": online,
            "batching_ratio": f.n_nodes / max(n_levels_main, 1),   # cells evaluated per batched step: Section 3's batching ratio at cell granularity
            "cpu_baseline": {"value": cpu_v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": cpu_sample,
                             "parallel_over_trees": cpu_par},
            "per_config": per_config,
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def launcher_command(n_ranks: int, argv, port: int):
    """The command that starts this script as `n_ranks` ranks of one node (what a driver would type itself)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="jdb", choices=["jdb", "reference"])
    ap.add_argument("--config", type=int, default=5, choices=[1, 2, 3, 4, 5],
                    help="workload of the top-level figures (default: the largest one, 5); the others go under per_config")
    ap.add_argument("--trees", type=int, default=None,
                    help="shrink the forest to this many trees of the same shape (profiler captures; not a bench value)")
    ap.add_argument("--mode", default="auto", choices=["auto", "level", "persistent"])
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of CPU time for each cpu_baseline sample")
    ap.add_argument("--all-configs", dest="all_configs", action="store_true", default=True,
                    help="also time the other four workloads and list them under per_config (1 GPU only)")
    ap.add_argument("--no-all-configs", dest="all_configs", action="store_false")
    ap.add_argument("--training-only", type=int, default=0, choices=[0, 1, 2, 3, 4, 5],
                    help="run only the training leg (fp32 forward + backward) of this workload and print its entry; "
                         "for profiling the backward kernels (honours --trees, --steps, --warmup)")
    ap.add_argument("--rendezvous-only", action="store_true",
                    help="start the ranks, reduce the totals over gloo on the CPU and print them: checks the launcher, times nothing")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started bare: become the launcher of the N ranks (rank 0 prints the line)
        raise SystemExit(subprocess.call(launcher_command(args.gpus, sys.argv[1:], free_port())))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
