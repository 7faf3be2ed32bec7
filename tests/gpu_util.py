"""Helpers for the GPU parity tests: move a workload to the device and run the C-ABI path on it."""
import os

import numpy as np
import torch

from paper_1904_07421_b200 import jdb
from paper_1904_07421_b200 import workloads as wl


def device_inputs(w: wl.Workload, pad_ld: bool = False):
    """(forest, x, packed, precision) on cuda:0.  x is gathered on the device from the table."""
    dev = torch.device("cuda:0")
    forest = jdb.forest_to_device(w.forest.child_ptr, w.forest.child_idx, dev)
    precision = jdb.BF16 if w.precision == "bf16" else jdb.FP32
    table = torch.from_numpy(w.table).to(dev)
    token = torch.from_numpy(w.token.astype(np.int64)).to(dev)
    dt = torch.bfloat16 if precision == jdb.BF16 else torch.float32
    n = max(forest.n_nodes, 1)
    ld = (w.D + 7) // 8 * 8 if pad_ld else w.D
    x = torch.zeros((n, ld), dtype=dt, device=dev)
    if forest.n_nodes:
        x[:forest.n_nodes, :w.D] = table.to(dt)[token]
    packed = jdb.jdb_pack_weights(torch.from_numpy(w.W).to(dev), torch.from_numpy(w.U).to(dev),
                                  torch.from_numpy(w.b).to(dev), precision)
    return forest, x, packed, precision


def padded_ldh(H: int) -> int:
    """Leading dimension of the padded output layout: a multiple of 4 floats, and never equal to H, so that there are
    always padding columns whose contents can be watched."""
    return (H + 4) // 4 * 4


def run_forward(w: wl.Workload, mode=jdb.MODE_AUTO, pad_ld=False, sync_schedule=True, flags=0, tuning=0, to_host=True,
                bench_ld=False):
    """bench_ld: the leading dimensions the benchmark uses (x rows padded to 8, h/c rows to 4 elements)."""
    flags |= int(os.environ.get("JDB_TEST_EXTRA_FLAGS", "0"))   # e.g. 2: the whole suite with the kernels' index checks on
    forest, x, packed, precision = device_inputs(w, pad_ld or bench_ld)
    sched = jdb.jdb_schedule(forest, sync=sync_schedule)
    ldh = (w.H + 3) // 4 * 4 if bench_ld else (padded_ldh(w.H) if pad_ld else w.H)
    n = max(forest.n_nodes, 1)
    h = torch.full((n, ldh), float("nan"), dtype=torch.float32, device=x.device)
    c = torch.full((n, ldh), float("nan"), dtype=torch.float32, device=x.device)
    jdb.jdb_treelstm_forward(forest, sched, x, packed, w.D, w.H, precision, mode=mode, h=h, c=c, flags=flags,
                             tuning=tuning)
    torch.cuda.synchronize()
    # the library promises not to write columns H .. ldh-1: the NaN canaries must still be there
    if ldh > w.H and forest.n_nodes:
        assert bool(torch.isnan(h[:, w.H:]).all()) and bool(torch.isnan(c[:, w.H:]).all()), "padding columns were written"
    if not to_host:
        return h[:forest.n_nodes, :w.H], c[:forest.n_nodes, :w.H], sched
    return h[:forest.n_nodes, :w.H].cpu().numpy(), c[:forest.n_nodes, :w.H].cpu().numpy(), sched


def level_structure(forest: wl.Forest):
    """(depth, perm, level_ptr) of a forest, computed here with whole-array numpy steps (height above the leaves by
    repeated propagation to the parents; ordering by a stable sort).  Used only to CHOOSE which trees a sampled test
    looks at; the expected values of those trees come from the CPU checker."""
    parent = wl.parent_array(forest)
    n = forest.n_nodes
    depth = np.zeros(n, dtype=np.int64)
    has_parent = parent >= 0
    while True:
        cand = np.zeros(n, dtype=np.int64)
        np.maximum.at(cand, parent[has_parent], depth[has_parent] + 1)
        new = np.maximum(depth, cand)
        if np.array_equal(new, depth):
            break
        depth = new
    perm = np.argsort(depth, kind="stable")
    level_ptr = np.concatenate([[0], np.cumsum(np.bincount(depth))])
    return depth, perm, level_ptr


def trees_of(forest: wl.Forest, nodes) -> np.ndarray:
    return np.unique(np.searchsorted(forest.tree_ptr, np.asarray(nodes, dtype=np.int64), side="right") - 1)


def deliberate_trees(forest: wl.Forest, row_bytes: int, extra_random: int, seed: int, tile: int = 128,
                     per_spot: int = 6) -> np.ndarray:
    """Trees a sampled parity test must not miss: the first and the last tree; the trees owning the rows around the
    boundary between leaves and internal nodes in level order; rows of the last (partial) tile of every level and
    of the first tile of the next; the rows on both sides of the points where a row's byte offset (by node id and
    by position in level order) passes 2^31 and 2^32; plus `extra_random` trees drawn at random."""
    depth, perm, level_ptr = level_structure(forest)
    n = forest.n_nodes
    spots = [0, n - 1]
    pos = []
    for l in range(1, len(level_ptr)):
        end = int(level_ptr[l])
        start_last_tile = end - ((end - int(level_ptr[l - 1]) - 1) % tile + 1)
        pos += list(range(max(start_last_tile, end - per_spot), end)) + list(range(start_last_tile, min(start_last_tile + 2, end)))
        pos += list(range(end, min(end + per_spot, n)))
    for shift in (31, 32):
        r = (1 << shift) // row_bytes
        for k in range(-2, 2):
            if 0 <= r + k < n:
                spots.append(r + k)
                pos.append(r + k)
    nodes = np.concatenate([np.asarray(spots, dtype=np.int64), perm[np.unique(np.asarray(pos, dtype=np.int64))]])
    rng = np.random.default_rng(seed)
    rnd = rng.choice(forest.n_trees, size=min(extra_random, forest.n_trees), replace=False)
    return np.unique(np.concatenate([trees_of(forest, nodes), rnd]))
