"""Parity of jdb_treelstm_backward (through the C ABI) with the per-node reverse-mode checker in fp64.

The backward pass computes in fp32; what separates it from the checker is fp32 rounding in the products, the order of
the sums over nodes and edges behind dW, dU and db (split over CTAs, added atomically) and the fp32 forward states
it is given.  Tolerance: 1e-4 relative to the largest entry of the block (the tolerance of the fp32 forward path).
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import treelstm_backward as ob
from paper_1904_07421_b200 import jdb
from paper_1904_07421_b200 import workloads as wl
from tests.gpu_util import padded_ldh

pytestmark = pytest.mark.gpu
TOL = 1e-4


def _close(got, ref, what):
    got = np.asarray(got, dtype=np.float64)
    scale = max(1.0, float(np.max(np.abs(ref))) if ref.size else 1.0)
    err = float(np.max(np.abs(got - ref))) if ref.size else 0.0
    assert np.all(np.isfinite(got)), what
    assert err <= TOL * scale, (what, err, scale)


def _run(w, gh, gc, pad=False, want_dx=True):
    """Forward (fp32) and backward on the device; returns host arrays."""
    dev = torch.device("cuda:0")
    f = w.forest
    forest = jdb.forest_to_device(f.child_ptr, f.child_idx, dev)
    sched = jdb.jdb_schedule(forest)
    n, D, H = f.n_nodes, w.D, w.H
    ldx = D + 3 if pad else D
    ldh = padded_ldh(H) if pad else H
    ldg = H + 5 if pad else H
    x = torch.full((max(n, 1), ldx), float("nan"), dtype=torch.float32, device=dev)
    if n:
        x[:n, :D] = torch.from_numpy(w.x_full()).to(dev)
    W, U, b = (torch.from_numpy(a).to(dev) for a in (w.W, w.U, w.b))
    packed = jdb.jdb_pack_weights(W, U, b, jdb.FP32)
    h = torch.full((max(n, 1), ldh), float("nan"), dtype=torch.float32, device=dev)
    c = torch.full((max(n, 1), ldh), float("nan"), dtype=torch.float32, device=dev)
    jdb.jdb_treelstm_forward(forest, sched, x, packed, D, H, jdb.FP32, h=h, c=c)
    g_h = torch.full((max(n, 1), ldg), float("nan"), dtype=torch.float32, device=dev)
    g_h[:n, :H] = torch.from_numpy(gh.astype(np.float32)).to(dev)
    g_c = None
    if gc is not None:
        g_c = torch.full((max(n, 1), ldg), float("nan"), dtype=torch.float32, device=dev)
        g_c[:n, :H] = torch.from_numpy(gc.astype(np.float32)).to(dev)
    dW, dU, db, dx = jdb.jdb_treelstm_backward(forest, sched, x, W, U, b, h, c, g_h, g_c, want_dx=want_dx)
    torch.cuda.synchronize()
    return dW.cpu().numpy(), dU.cpu().numpy(), db.cpu().numpy(), (dx.cpu().numpy() if want_dx else None)


def _check(w, gh, gc, **kw):
    f = w.forest
    got = _run(w, gh, gc, **kw)
    ref = ob.backward(f.child_ptr, f.child_idx, w.x_full(), w.W, w.U, w.b, gh.astype(np.float32), None if gc is None else gc.astype(np.float32))
    for name, g, r in zip(("dW", "dU", "db", "dx"), got, ref):
        if g is not None:
            _close(g, r, name)


def _grads(n, H, seed, with_c=True):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n, H)), (rng.standard_normal((n, H)) * 0.5 if with_c else None)


@pytest.mark.parametrize("D,H", [(3, 2), (5, 7), (16, 40), (64, 64)])
@pytest.mark.parametrize("pad", [False, True])
def test_small_forests_every_block(D, H, pad):
    """0 to 3 children per node, a chain, lone nodes; odd sizes take the element-wise loads, padded rows the strides."""
    parents = [[-1, 0, 0, 1, 1, 1, 2], [-1, 0, 1, 2, 3], [-1], [-1, 0], [-1]]
    w = wl.make_custom(parents, D=D, H=H, seed=31 + D, bias="random")
    gh, gc = _grads(w.forest.n_nodes, H, 7)
    _check(w, gh, gc, pad=pad)


def test_no_grad_c_and_no_dx():
    w = wl.make_custom([[-1, 0, 0, 2], [-1, 0]], D=8, H=12, seed=3, bias="random")
    gh, _ = _grads(w.forest.n_nodes, 12, 9, with_c=False)
    _check(w, gh, None, want_dx=False)


def test_loss_on_the_roots_only():
    """The usual training case: only root states enter the loss."""
    w = dataclasses.replace(wl.make_workload(1, n_trees=40, bias="random"), precision="fp32")
    f = w.forest
    gh, _ = _grads(f.n_nodes, w.H, 11, with_c=False)
    roots = np.asarray(f.tree_ptr[:-1], dtype=np.int64)
    mask = np.zeros(f.n_nodes, dtype=bool)
    mask[roots] = True
    gh[~mask] = 0.0
    _check(w, gh, None)


@pytest.mark.parametrize("index,n_trees", [(1, 200), (2, 120), (3, 60), (4, 12), (5, 60)])
def test_workload_shapes_shrunk(index, n_trees):
    """The five forest shapes at sizes the checker finishes in seconds, D and H cut so that several 128-row tiles and a
    ragged tail appear in every product (rows: nodes, edges; columns: 4H = 160 and H = 40)."""
    base = wl.make_workload(index, n_trees=n_trees, bias="random")
    w = wl.make_custom([[-1]], D=24, H=40, seed=index, bias="random")
    rng = np.random.default_rng(100 + index)
    token = rng.integers(0, w.table.shape[0], size=base.forest.n_nodes).astype(np.int32)
    w = dataclasses.replace(w, forest=base.forest, token=token)
    gh, gc = _grads(base.forest.n_nodes, 40, 13 + index)
    _check(w, gh, gc)


def test_wide_fan_out_and_relabelled_ids():
    """A root with 140 children beside deep chains, node ids shuffled (ids are not in topological order)."""
    deep = [-1] + list(range(60))
    parents = [[-1] + [0] * 140, deep, [-1, 0, 0, 1, 1, 2, 2]]
    w = wl.make_custom(parents, D=16, H=24, seed=17, bias="random")
    forest, _ = wl.relabel(w.forest, np.random.default_rng(5))
    w = dataclasses.replace(w, forest=forest)
    gh, gc = _grads(forest.n_nodes, 24, 19)
    _check(w, gh, gc)


def test_gradient_of_some_trees_equals_the_subforest():
    """A forest too large for the checker as a whole: with the loss on a sample of trees only, every other node's
    gradient is zero, so dW, dU and db equal the checker's on the sub-forest of the sample, and dx its rows there (zero
    elsewhere)."""
    w = dataclasses.replace(wl.make_workload(3, n_trees=600, bias="random"), precision="fp32")
    w = dataclasses.replace(w, D=48, H=72, table=w.table[:, :48].copy(),
                            W=np.ascontiguousarray(np.concatenate([w.W[g * w.H:g * w.H + 72, :48] for g in range(4)])),
                            U=np.ascontiguousarray(np.concatenate([w.U[g * w.H:g * w.H + 72, :72] for g in range(4)])),
                            b=np.ascontiguousarray(np.concatenate([w.b[g * w.H:g * w.H + 72] for g in range(4)])))
    f = w.forest
    rng = np.random.default_rng(23)
    trees = np.unique(np.concatenate([[0, f.n_trees - 1], rng.choice(f.n_trees, size=25, replace=False)]))
    sub, nodes = wl.subforest(f, trees)
    gh = np.zeros((f.n_nodes, w.H))
    gc = np.zeros((f.n_nodes, w.H))
    gh[nodes] = rng.standard_normal((len(nodes), w.H))
    gc[nodes] = rng.standard_normal((len(nodes), w.H)) * 0.5
    dW, dU, db, dx = _run(w, gh, gc)
    ref = ob.backward(sub.child_ptr, sub.child_idx, w.x_rows(nodes), w.W, w.U, w.b, gh[nodes].astype(np.float32), gc[nodes].astype(np.float32))
    _close(dW, ref[0], "dW")
    _close(dU, ref[1], "dU")
    _close(db, ref[2], "db")
    _close(dx[nodes], ref[3], "dx")
    others = np.setdiff1d(np.arange(f.n_nodes), nodes)
    assert np.all(dx[others] == 0.0)


def test_large_forest_sampled_trees():
    """Workload 5's shape at 12288 trees (about 290 k nodes, D = H = 1024): the gradient rows of the workspace pass the
    2^31 and 2^32 byte offsets, the edge-slot scan spans several hundred blocks, the parameter gradients split their
    contraction many ways.  Loss on a sample of trees (the first, the last, the owners of the rows at those offsets and
    random ones); the checker runs on their sub-forest (about 10 s)."""
    w = dataclasses.replace(wl.make_workload(5, n_trees=12288, bias="random"), precision="fp32")
    f = w.forest
    rng = np.random.default_rng(29)
    rows = [0, f.n_nodes - 1] + [(1 << s) // (4 * 4 * w.H) + k for s in (31, 32) for k in (-1, 0, 1)]
    trees = np.unique(np.concatenate([np.searchsorted(f.tree_ptr, np.asarray(rows), side="right") - 1,
                                      rng.choice(f.n_trees, size=6, replace=False)]))
    sub, nodes = wl.subforest(f, trees)
    gh = np.zeros((f.n_nodes, w.H), dtype=np.float32)
    gc = np.zeros((f.n_nodes, w.H), dtype=np.float32)
    gh[nodes] = rng.standard_normal((len(nodes), w.H))
    gc[nodes] = rng.standard_normal((len(nodes), w.H)) * 0.5
    dW, dU, db, dx = _run(w, gh, gc)
    ref = ob.backward(sub.child_ptr, sub.child_idx, w.x_rows(nodes), w.W, w.U, w.b, gh[nodes], gc[nodes])
    _close(dW, ref[0], "dW")
    _close(dU, ref[1], "dU")
    _close(db, ref[2], "db")
    _close(dx[nodes], ref[3], "dx")
    mask = np.ones(f.n_nodes, dtype=bool)
    mask[nodes] = False
    assert not dx[mask].any()


def test_empty_forest_and_argument_errors():
    dev = torch.device("cuda:0")
    a = wl.make_custom([[-1, 0, 0, 1]], D=4, H=4, seed=1)
    W, U, b = (torch.from_numpy(t).to(dev) for t in (a.W, a.U, a.b))
    z = torch.zeros((4, 4), device=dev)
    empty = jdb.forest_to_device([0], [])
    dW, dU, db, dx = jdb.jdb_treelstm_backward(empty, jdb.jdb_schedule(empty), z, W, U, b, z, z.clone(), z.clone())
    torch.cuda.synchronize()
    assert not bool(dW.any()) and not bool(dU.any()) and not bool(db.any()) and dx.shape[0] == 0
    # the level table is needed on the host: a schedule whose counts were never read back is refused
    fa = jdb.forest_to_device(a.forest.child_ptr, a.forest.child_idx, dev)
    with pytest.raises(jdb.JdbError):
        jdb.jdb_treelstm_backward(fa, jdb.jdb_schedule(fa, sync=False), z, W, U, b, z, z.clone(), z.clone())
    # a workspace that is too small
    with pytest.raises(jdb.JdbError):
        jdb.jdb_treelstm_backward(fa, jdb.jdb_schedule(fa), z, W, U, b, z, z.clone(), z.clone(),
                                  ws=torch.empty(256, dtype=torch.uint8, device=dev))
