"""jdb_schedule_static: the analysis for callers that cannot allocate a workspace.

Collected last on purpose.  The entry point keeps its scratch in a fixed array inside the library, so the test
checks what such a caller relies on: it gives the same schedule as jdb_schedule, twice in a row on the shared
array (the second call must not see the first one's leftovers), it refuses forests beyond its limit, and the
caching allocator is not touched while it runs.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_1904_07421_b200 import jdb
from paper_1904_07421_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _compare(forest, a, b):
    n = forest.n_nodes
    assert a.n_levels == b.n_levels and a.n_leaves == b.n_leaves
    assert torch.equal(a.depth[:n], b.depth[:n])
    assert torch.equal(a.perm[:n], b.perm[:n])
    assert torch.equal(a.level_ptr[:a.n_levels + 1], b.level_ptr[:b.n_levels + 1])


def test_static_scratch_schedule_matches_the_workspace_one_twice():
    # two different forests, both beyond the one-CTA path so that the scratch array is really used
    w1 = wl.make_workload(3, n_trees=500)
    w2, _ = wl.relabel(wl.make_workload(4, n_trees=40).forest, np.random.default_rng(12))
    f1 = jdb.forest_to_device(w1.forest.child_ptr, w1.forest.child_idx)
    f2 = jdb.forest_to_device(w2.child_ptr, w2.child_idx)
    assert 6144 < f1.n_nodes <= jdb.STATIC_MAX_NODES and 6144 < f2.n_nodes <= jdb.STATIC_MAX_NODES
    ref1, ref2 = jdb.jdb_schedule(f1), jdb.jdb_schedule(f2)
    out1, out2 = jdb.alloc_schedule(f1.n_nodes), jdb.alloc_schedule(f2.n_nodes)
    torch.cuda.synchronize()
    before = torch.cuda.memory_stats()["allocation.all.allocated"]
    jdb.jdb_schedule_static(f1, out1)      # first call on this device: looks the scratch address up
    jdb.jdb_schedule_static(f2, out2)      # second call, same scratch, different forest
    jdb.jdb_schedule_static(f1, out1)      # and back again
    torch.cuda.synchronize()
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == before
    _compare(f1, out1, ref1)
    _compare(f2, out2, ref2)
    # and directly against the CPU checker, so that this entry point does not lean on the other one being right
    from oracle import schedule as osched
    for forest_np, out in ((w1.forest, out1), (w2, out2)):
        depth, level_ptr, perm, _, n_levels = osched.schedule(forest_np.child_ptr, forest_np.child_idx, forest_np.n_nodes)
        assert out.n_levels == n_levels
        assert np.array_equal(out.depth.cpu().numpy(), depth) and np.array_equal(out.perm.cpu().numpy(), perm)
        assert np.array_equal(out.level_ptr[:n_levels + 1].cpu().numpy(), level_ptr)


def test_static_scratch_schedule_limits_and_errors():
    n = jdb.STATIC_MAX_NODES + 1
    big = jdb.forest_to_device(np.zeros(n + 1, dtype=np.int32), np.zeros(0, dtype=np.int32))
    with pytest.raises(jdb.JdbError) as ei:
        jdb.jdb_schedule_static(big)
    assert ei.value.status == jdb.ERR_UNSUPPORTED
    # a malformed forest is reported, and a good one still works afterwards
    cp = np.arange(0, 8001, dtype=np.int32)                # every node has one child ...
    ci = np.roll(np.arange(8000, dtype=np.int32), 1)      # ... its predecessor: one big cycle
    with pytest.raises(jdb.JdbError) as ei:
        jdb.jdb_schedule_static(jdb.forest_to_device(cp, ci))
    assert ei.value.status == jdb.ERR_NOT_A_FOREST
    w = wl.make_workload(2)
    f = jdb.forest_to_device(w.forest.child_ptr, w.forest.child_idx)
    _compare(f, jdb.jdb_schedule_static(f), jdb.jdb_schedule(f))
    L = jdb.lib()
    assert L.jdb_schedule_static(None, None, None) == jdb.ERR_INVALID_ARG
