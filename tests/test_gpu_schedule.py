"""GPU batching analysis vs the CPU checker: depth, level_ptr, perm must match bit for bit."""
import numpy as np
import pytest
import torch

from conftest import read_golden
from oracle import schedule as osched
from paper_1904_07421_b200 import jdb
from paper_1904_07421_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def gpu_schedule(child_ptr, child_idx, sync=True):
    forest = jdb.forest_to_device(np.asarray(child_ptr, dtype=np.int32), np.asarray(child_idx, dtype=np.int32))
    s = jdb.jdb_schedule(forest, sync=sync)
    torch.cuda.synchronize()
    return forest, s


def assert_matches_oracle(child_ptr, child_idx):
    n = len(child_ptr) - 1
    depth, level_ptr, perm, _, n_levels = osched.schedule(child_ptr, child_idx, n)
    forest, s = gpu_schedule(child_ptr, child_idx)
    assert s.n_levels == n_levels
    assert s.n_leaves == (int(level_ptr[1]) if n_levels > 0 else 0)
    assert np.array_equal(s.level_ptr[:n_levels + 1].cpu().numpy(), level_ptr)
    if n:
        assert np.array_equal(s.depth[:n].cpu().numpy(), depth)
        assert np.array_equal(s.perm[:n].cpu().numpy(), perm)
    meta = s.meta.cpu().numpy()
    assert meta[0] == n_levels and meta[1] == 0 and meta[4] == 0
    # leading run of levels 1, 2, ... holding at least 65536 nodes (the forward pass launches those on their own)
    sizes = np.diff(np.asarray(level_ptr))[1:]
    wide = 0
    while wide < len(sizes) and sizes[wide] >= 65536:
        wide += 1
    assert s.n_wide_levels == wide and meta[7] == wide
    return s


def test_worked_example():
    g = read_golden("forest10.txt")
    s = assert_matches_oracle(g["child_ptr"], g["child_idx"])
    assert s.perm[:10].cpu().tolist() == g["perm"]  # and directly against the hand-made table
    assert s.depth[:10].cpu().tolist() == g["depth"]


def test_empty_single_chain_star():
    assert_matches_oracle([0], [])
    assert_matches_oracle([0, 0], [])
    n = 300
    f = wl.forest_from_global_parent(np.array([-1] + list(range(n - 1))))
    assert_matches_oracle(f.child_ptr, f.child_idx)
    f = wl.forest_from_global_parent(np.array([-1] + [0] * (n - 1)))
    assert_matches_oracle(f.child_ptr, f.child_idx)


def test_random_relabelled_small_forests():
    rng = np.random.default_rng(3)
    for trial in range(25):
        n = int(rng.integers(1, 400))
        parent = np.full(n, -1, dtype=np.int64)
        for v in range(1, n):
            if rng.random() < 0.9:
                parent[v] = rng.integers(max(0, v - 12), v)
        f, _ = wl.relabel(wl.forest_from_global_parent(parent), rng)
        assert_matches_oracle(f.child_ptr, f.child_idx)


@pytest.mark.parametrize("index", [1, 2, 3, 4, 5])
def test_workload_forests_bit_exact(index):
    w = wl.make_workload(index)
    assert_matches_oracle(w.forest.child_ptr, w.forest.child_idx)


def test_relabelled_large_forest_general_path():
    w = wl.make_workload(3, n_trees=600)
    f, _ = wl.relabel(w.forest, np.random.default_rng(1))
    assert f.n_nodes > 6144
    assert_matches_oracle(f.child_ptr, f.child_idx)


def test_more_than_2048_levels_needs_two_sort_passes():
    n = 9000  # a chain of 5000 next to smaller trees: n_levels = 5000 > 2^11
    parent = np.full(n, -1, dtype=np.int64)
    parent[1:5000] = np.arange(0, 4999)
    rng = np.random.default_rng(2)
    for v in range(5001, n):
        parent[v] = rng.integers(5000, v)
    f, _ = wl.relabel(wl.forest_from_global_parent(parent), rng)
    s = assert_matches_oracle(f.child_ptr, f.child_idx)
    assert s.n_levels == 5000


def test_deep_small_forest_one_cta_path():
    n = 6000  # fits the one-CTA path; 4000 levels squeeze its rank counters
    parent = np.full(n, -1, dtype=np.int64)
    parent[1:4000] = np.arange(0, 3999)
    parent[4001:] = 4000
    f, _ = wl.relabel(wl.forest_from_global_parent(parent), np.random.default_rng(4))
    assert_matches_oracle(f.child_ptr, f.child_idx)


def test_async_schedule_leaves_counts_on_device():
    w = wl.make_workload(2)
    forest, s = gpu_schedule(w.forest.child_ptr, w.forest.child_idx, sync=False)
    assert s.n_levels == -1 and s.n_leaves == -1
    depth, level_ptr, perm, _, n_levels = osched.schedule(w.forest.child_ptr, w.forest.child_idx, w.forest.n_nodes)
    meta = s.meta.cpu().numpy()
    assert meta[0] == n_levels and meta[3] == level_ptr[1]
    assert np.array_equal(s.perm.cpu().numpy(), perm)


def _csr(n, edges):
    """CSR of n nodes from (parent, child) pairs; children keep the order of the list."""
    cp = np.zeros(n + 1, dtype=np.int64)
    for p, _ in edges:
        cp[p + 1] += 1
    cp = np.cumsum(cp)
    ci = np.array([c for _, c in sorted(edges, key=lambda e: e[0])], dtype=np.int32)
    return cp.astype(np.int32), ci


@pytest.mark.parametrize("big", [False, True])
@pytest.mark.parametrize("kind", ["range", "negative", "two_parents", "cycle", "self_loop", "bad_ptr"])
def test_malformed_forest_is_reported_not_faulted(kind, big):
    n = 7000 if big else 50   # both the one-CTA path and the general path
    edges = [((v - 1) // 2, v) for v in range(1, n)]
    good_cp, good_ci = _csr(n, edges)
    if kind == "cycle":
        edges[0] = (3, 1)          # 1 -> 3 -> 1: every node still has at most one parent
    elif kind == "self_loop":
        edges[0] = (1, 1)
    cp, ci = _csr(n, edges)
    if kind == "range":
        ci[5] = n + 3
    elif kind == "negative":
        ci[5] = -2
    elif kind == "two_parents":
        ci[5] = ci[6]
    elif kind == "bad_ptr":
        cp[4] = cp[5] + 1
    with pytest.raises(osched.NotAForest):
        osched.schedule(cp, ci, n)
    forest = jdb.forest_to_device(cp, ci)
    with pytest.raises(jdb.JdbError) as ei:
        jdb.jdb_schedule(forest)
    assert ei.value.status == jdb.ERR_NOT_A_FOREST
    assert_matches_oracle(good_cp, good_ci)   # the context is still healthy


def test_argument_errors():
    forest = jdb.forest_to_device([0, 1, 1], [1])
    s = jdb.alloc_schedule(2)
    cf, cs = forest.c(), s.c()
    import ctypes as C
    L = jdb.lib()
    assert L.jdb_schedule(None, C.byref(cs), None, 0, None) == jdb.ERR_INVALID_ARG
    assert L.jdb_schedule(C.byref(cf), None, None, 0, None) == jdb.ERR_INVALID_ARG
    big = jdb.forest_to_device(np.zeros(10001, dtype=np.int32), np.zeros(0, dtype=np.int32))
    sb = jdb.alloc_schedule(10000)
    cfb, csb = big.c(), sb.c()
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    assert L.jdb_schedule(C.byref(cfb), C.byref(csb), C.c_void_p(ws.data_ptr()), 1024, None) == jdb.ERR_WORKSPACE


@pytest.mark.parametrize("index", [1, 2, 3, 4, 5])
def test_launch_counts_match_the_checker(index):
    """Section 3's launch counts at cell and at operator granularity: the GPU count of distinct (depth, number of
    children) pairs against the one-node-at-a-time checker, on the five workloads and on the hand-counted forest."""
    from oracle import granularity as og
    f = wl.make_workload(index).forest
    forest, s = gpu_schedule(f.child_ptr, f.child_idx)
    got = jdb.jdb_launch_counts(forest, s)
    depth = s.depth[:f.n_nodes].cpu().numpy()            # bit-exact against the checker's depths elsewhere in this file
    assert got == og.launch_counts(f.child_ptr, depth)
    if index == 1:
        g = read_golden("forest10.txt")
        forest, s = gpu_schedule(g["child_ptr"], g["child_idx"])
        assert list(jdb.jdb_launch_counts(forest, s)) == g["launch_counts"]
        empty, se = gpu_schedule([0], [])
        assert jdb.jdb_launch_counts(empty, se) == (0, 0, 0, 0, 0)
