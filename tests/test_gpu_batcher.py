"""The table of slots by (depth, key) and the execution of forests of two kinds of cells, through the C ABI, against
oracle/batcher.py: the table bit for bit, h and c within 1e-4 (fp32 products and sums, as the fp32 forward path)."""
import numpy as np
import pytest
import torch

from oracle import batcher as ob
from paper_1904_07421_b200 import jdb
from paper_1904_07421_b200 import workloads as wl

pytestmark = pytest.mark.gpu
TOL = 1e-4
DEV = "cuda:0"


def _plan(f, key, n_keys):
    forest = jdb.forest_to_device(f.child_ptr, f.child_idx, DEV)
    sched = jdb.jdb_schedule(forest)
    plan = jdb.jdb_batch_plan(forest, sched, torch.from_numpy(np.asarray(key, dtype=np.int32)).to(DEV), n_keys)
    return forest, sched, plan


def _check_plan(f, key, n_keys):
    forest, sched, plan = _plan(f, key, n_keys)
    perm, slot_ptr, slot_depth, slot_key, _ = ob.plan(f.child_ptr, f.child_idx, key)
    S = len(slot_depth)
    assert plan.n_slots == S
    assert np.array_equal(plan.perm[:f.n_nodes].cpu().numpy(), perm)
    assert np.array_equal(plan.slot_ptr[:S + 1].cpu().numpy(), slot_ptr)
    assert np.array_equal(plan.slot_depth[:S].cpu().numpy(), slot_depth)
    assert np.array_equal(plan.slot_key[:S].cpu().numpy(), slot_key)
    return forest, sched, plan


@pytest.mark.parametrize("index,n_trees,n_keys", [(1, 64, 2), (2, 256, 5), (3, 700, 3), (4, 40, 300), (5, 3000, 2)])
def test_table_is_bit_exact(index, n_trees, n_keys):
    """All five forest shapes; sizes cross several sort tiles (2048) and scan blocks (1024) with ragged tails, and the
    sort key needs one, two or three 8-bit passes (13 levels x 3 keys ... 87 levels x 300 keys)."""
    rng = np.random.default_rng(40 + index)
    f = wl.make_forest(index, rng, n_trees=n_trees)
    _check_plan(f, rng.integers(0, n_keys, size=f.n_nodes), n_keys)


def test_table_at_full_size():
    """Workload 5's whole forest (1.57 M nodes): 1535 scan blocks (the scanning CTA walks its block sums in two rounds)
    and 768 sort tiles."""
    rng = np.random.default_rng(77)
    f = wl.make_forest(5, rng)
    _check_plan(f, rng.integers(0, 3, size=f.n_nodes), 3)


def test_table_edge_cases():
    one = wl.forest_from_parents([np.asarray([-1])])
    _check_plan(one, [0], 1)
    chain = wl.forest_from_parents([np.asarray([-1] + list(range(2500)))])      # one node per slot
    _check_plan(chain, np.arange(2501) % 2, 2)
    flat = wl.forest_from_parents([np.asarray([-1])] * 5000)                     # one level, one key: one slot
    _check_plan(flat, np.zeros(5000, dtype=int), 7)
    empty = jdb.forest_to_device([0], [])
    plan = jdb.jdb_batch_plan(empty, jdb.jdb_schedule(empty), torch.zeros(1, dtype=torch.int32, device=DEV), 3)
    assert plan.n_slots == 0 and int(plan.slot_ptr[0]) == 0
    f = wl.forest_from_parents([np.asarray([-1, 0, 0])])
    with pytest.raises(jdb.JdbError):
        _plan(f, [0, 5, 1], 2)                                                    # key out of range
    forest = jdb.forest_to_device(f.child_ptr, f.child_idx, DEV)
    with pytest.raises(jdb.JdbError):                                             # level count never read back
        jdb.jdb_batch_plan(forest, jdb.jdb_schedule(forest, sync=False), torch.zeros(3, dtype=torch.int32, device=DEV), 2)


def _cells(rng, D, H, kinds):
    host, dev = [], []
    for kind, arity in kinds:
        W, U, b = wl.make_weights(rng, D, H, "normal", "random")
        if kind == "nary":
            U = (rng.standard_normal(((3 + arity) * H, arity * H)) / np.sqrt(arity * H)).astype(np.float32)
        host.append(dict(kind=kind, arity=arity, W=W, U=U, b=b))
        dev.append((jdb.CELL_NARY if kind == "nary" else jdb.CELL_CHILDSUM, arity,
                    *(torch.from_numpy(a).to(DEV) for a in (W, U, b))))
    return host, dev


def _check_forward(f, key, kinds, D, H, seed, pad=False):
    rng = np.random.default_rng(seed)
    host, dev = _cells(rng, D, H, kinds)
    x = rng.standard_normal((f.n_nodes, D)).astype(np.float32)
    forest, sched, plan = _plan(f, key, len(kinds))
    ldx, ldh = (D + 3, H + 5) if pad else (D, H)
    xd = torch.full((f.n_nodes, ldx), float("nan"), device=DEV)
    xd[:, :D] = torch.from_numpy(x).to(DEV)
    h = torch.full((f.n_nodes, ldh), float("nan"), device=DEV)
    c = torch.full((f.n_nodes, ldh), float("nan"), device=DEV)
    kd = torch.from_numpy(np.asarray(key, dtype=np.int32)).to(DEV)
    jdb.jdb_cells_forward(forest, plan, kd, dev, xd, D, H, h=h, c=c)
    torch.cuda.synchronize()
    ho, co = ob.forward_mixed(f.child_ptr, f.child_idx, x, key, host)
    hg, cg = h[:, :H].cpu().numpy(), c[:, :H].cpu().numpy()
    assert np.all(np.isfinite(hg)) and np.all(np.isfinite(cg))
    assert np.max(np.abs(hg - ho)) <= TOL and np.max(np.abs(cg - co)) <= TOL
    if pad:
        assert bool(torch.isnan(h[:, H:]).all()) and bool(torch.isnan(c[:, H:]).all()), "padding columns were written"
    return forest, sched, hg, cg, x, host


@pytest.mark.parametrize("D,H,pad", [(3, 2, False), (5, 7, True), (24, 40, False), (64, 64, True)])
def test_two_kinds_of_cells_in_one_forest(D, H, pad):
    """Binary trees whose nodes are Child-Sum or binary N-ary cells at random; odd sizes, padded rows."""
    rng = np.random.default_rng(D)
    f = wl.forest_from_parents(wl._trees_capped(rng, 60, 3, 40, 2))
    key = rng.integers(0, 2, size=f.n_nodes)
    _check_forward(f, key, [("childsum", 0), ("nary", 2)], D, H, seed=D + 1, pad=pad)


def test_three_cells_and_arity_three():
    rng = np.random.default_rng(8)
    f = wl.forest_from_parents(wl._trees_capped(rng, 300, 5, 60, 3))
    key = rng.integers(0, 3, size=f.n_nodes)
    _check_forward(f, key, [("nary", 3), ("childsum", 0), ("nary", 3)], 20, 24, seed=2)


def test_child_sum_only_equals_the_forward_pass():
    """With one Child-Sum cell the executor computes what jdb_treelstm_forward computes (fp32): same values to 1e-5, on a
    forest with fan-outs up to 8 and 140."""
    wide = wl.forest_from_parents(list(wl._trees_capped(np.random.default_rng(1), 50, 10, 60, 8)) + [np.asarray([-1] + [0] * 140)])
    D, H = 32, 48
    key = np.zeros(wide.n_nodes, dtype=int)
    forest, sched, hg, cg, x, host = _check_forward(wide, key, [("childsum", 0)], D, H, seed=5)
    W, U, b = (torch.from_numpy(host[0][k]).to(DEV) for k in ("W", "U", "b"))
    packed = jdb.jdb_pack_weights(W, U, b, jdb.FP32)
    h2, c2 = jdb.jdb_treelstm_forward(forest, sched, torch.from_numpy(x).to(DEV), packed, D, H, jdb.FP32)
    torch.cuda.synchronize()
    assert np.max(np.abs(h2.cpu().numpy() - hg)) <= 1e-5 and np.max(np.abs(c2.cpu().numpy() - cg)) <= 1e-5


def test_too_many_children_is_refused():
    f = wl.forest_from_parents([np.asarray([-1, 0, 0, 0])])
    rng = np.random.default_rng(1)
    host, dev = _cells(rng, 4, 4, [("nary", 2)])
    forest, sched, plan = _plan(f, [0, 0, 0, 0], 1)
    with pytest.raises(jdb.JdbError):
        jdb.jdb_cells_forward(forest, plan, torch.zeros(4, dtype=torch.int32, device=DEV), dev, torch.zeros((4, 4), device=DEV), 4, 4)
