"""Pins for oracle/batcher.py: the table of slots by (depth, key) and the forest of two kinds of cells."""
import itertools
import math
import os

import numpy as np
import torch

from oracle import batcher as ob
from oracle import schedule as osched
from oracle import treelstm as ot
from paper_1904_07421_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        if line.startswith("#") or ":" not in line:
            continue
        k, v = line.split(":")
        out[k.strip()] = np.asarray([int(t) for t in v.split()], dtype=np.int64)
    return out


def test_hand_made_table():
    g, f = _read("plan10.txt"), _read("forest10.txt")
    perm, slot_ptr, slot_depth, slot_key, depth = ob.plan(f["child_ptr"], f["child_idx"], g["key"])
    assert np.array_equal(depth, f["depth"])
    for name, got in (("perm", perm), ("slot_ptr", slot_ptr), ("slot_depth", slot_depth), ("slot_key", slot_key)):
        assert np.array_equal(got, g[name]), name


def test_one_key_is_the_depth_table():
    for index in (1, 2, 4):
        f = wl.make_forest(index, np.random.default_rng(index), n_trees=20)
        depth, level_ptr, perm, _, n_levels = osched.schedule(f.child_ptr, f.child_idx, f.n_nodes)
        p, sp, sd, sk, _ = ob.plan(f.child_ptr, f.child_idx, np.full(f.n_nodes, 3))
        assert np.array_equal(p, perm) and np.array_equal(sp, level_ptr[:n_levels + 1])
        assert np.array_equal(sd, np.arange(n_levels)) and np.all(sk == 3)


def test_table_against_a_plain_sort_and_its_invariants():
    rng = np.random.default_rng(4)
    for index in (1, 3, 5):
        f = wl.make_forest(index, rng, n_trees=30)
        n = f.n_nodes
        key = rng.integers(0, 4, size=n)
        perm, slot_ptr, slot_depth, slot_key, depth = ob.plan(f.child_ptr, f.child_idx, key)
        assert list(perm) == sorted(range(n), key=lambda v: (depth[v], key[v], v))          # brute force
        assert sorted(perm) == list(range(n)) and slot_ptr[0] == 0 and slot_ptr[-1] == n
        pairs = list(zip(slot_depth, slot_key))
        assert pairs == sorted(set(zip(depth, key)))                                        # one slot per pair, in order
        parent = wl.parent_array(f)
        slot_of = np.empty(n, dtype=np.int64)
        for s in range(len(pairs)):
            members = perm[slot_ptr[s]:slot_ptr[s + 1]]
            assert len(members) > 0 and np.all(depth[members] == slot_depth[s]) and np.all(key[members] == slot_key[s])
            slot_of[members] = s
        has = parent >= 0
        assert np.all(slot_of[parent[has]] > slot_of[has])      # a node's slot runs after the slots of its children


def _tied(W, U, b, arity):
    """N-ary weights that make the cell a Child-Sum cell: the same U_iou for every position, U_f on the diagonal."""
    H = U.shape[1]
    Un = np.zeros(((3 + arity) * H, arity * H))
    for l in range(arity):
        Un[:3 * H, l * H:(l + 1) * H] = U[:3 * H]
        Un[(3 + l) * H:(4 + l) * H, l * H:(l + 1) * H] = U[3 * H:]
    return dict(kind="nary", arity=arity, W=W, U=Un, b=b)


def test_nary_with_tied_weights_is_the_child_sum_cell():
    for arity, cap in ((2, 2), (3, 3), (4, 2)):
        rng = np.random.default_rng(arity)
        trees = wl._trees_capped(rng, 12, 3, 25, cap)
        f = wl.forest_from_parents(trees)
        W, U, b = wl.make_weights(rng, 5, 4, "normal", "random")
        x = rng.standard_normal((f.n_nodes, 5))
        h0, c0 = ot.forward(f.child_ptr, f.child_idx, x, W, U, b)
        h1, c1 = ob.forward_mixed(f.child_ptr, f.child_idx, x, np.zeros(f.n_nodes, dtype=int), [_tied(W, U, b, arity)])
        assert np.max(np.abs(h0 - h1)) < 1e-13 and np.max(np.abs(c0 - c1)) < 1e-13
        # and the Child-Sum branch of the mixed evaluator is the Child-Sum checker itself
        h2, c2 = ob.forward_mixed(f.child_ptr, f.child_idx, x, np.zeros(f.n_nodes, dtype=int), [dict(kind="childsum", W=W, U=U, b=b)])
        assert np.max(np.abs(h0 - h2)) < 1e-13 and np.max(np.abs(c0 - c2)) < 1e-13


def test_unary_chain_is_a_library_lstm():
    T, D, H = 6, 3, 4
    rng = np.random.default_rng(2)
    f = wl.forest_from_parents([np.asarray([-1] + list(range(T - 1)))])
    W, U, b = wl.make_weights(rng, D, H, "normal", "random")
    x = rng.standard_normal((T, D))
    cell = dict(kind="nary", arity=1, W=W, U=U, b=b)          # arity 1: U is [4H, H] in blocks (i, o, u, f_1)
    h, c = ob.forward_mixed(f.child_ptr, f.child_idx, x, np.zeros(T, dtype=int), [cell])
    lstm = torch.nn.LSTMCell(D, H, bias=True, dtype=torch.float64)
    order = [0, 3, 2, 1]                                        # torch: (input, forget, cell, output)
    blk = lambda M: torch.cat([torch.from_numpy(np.asarray(M, dtype=np.float64)[g * H:(g + 1) * H]) for g in order])
    with torch.no_grad():
        lstm.weight_ih.copy_(blk(W)); lstm.weight_hh.copy_(blk(U)); lstm.bias_ih.copy_(blk(b)); lstm.bias_hh.zero_()
        hs, cs = torch.zeros(1, H, dtype=torch.float64), torch.zeros(1, H, dtype=torch.float64)
        for t in range(T - 1, -1, -1):                          # node t's only child is node t + 1
            hs, cs = lstm(torch.from_numpy(x[t:t + 1]), (hs, cs))
            assert np.max(np.abs(hs.numpy()[0] - h[t])) < 1e-12 and np.max(np.abs(cs.numpy()[0] - c[t])) < 1e-12


def test_scalar_binary_cell_worked_by_hand():
    """H = D = 1, two leaf children.  Only U_f^12 is non-zero among the forget blocks, so f_1 sees h_2 and f_2 sees no
    child at all: an implementation that swaps k and l, or sums the wrong block, lands elsewhere."""
    sg = lambda t: 1.0 / (1.0 + math.exp(-t))
    wi, wo, wu, wf = 0.3, -0.2, 0.5, 0.1
    bi, bo, bu, bf = 0.05, 0.1, -0.1, 0.2
    ui1, ui2, uo1, uo2, uu1, uu2 = 0.7, -0.4, 0.2, 0.6, -0.5, 0.9
    u12 = 1.5
    x0, x1, x2 = 0.8, -1.1, 0.6
    leaf = lambda x: (sg(wo * x + bo) * math.tanh(sg(wi * x + bi) * math.tanh(wu * x + bu)), sg(wi * x + bi) * math.tanh(wu * x + bu))
    (h1, c1), (h2, c2) = leaf(x1), leaf(x2)
    i = sg(wi * x0 + ui1 * h1 + ui2 * h2 + bi)
    o = sg(wo * x0 + uo1 * h1 + uo2 * h2 + bo)
    u = math.tanh(wu * x0 + uu1 * h1 + uu2 * h2 + bu)
    f1, f2 = sg(wf * x0 + u12 * h2 + bf), sg(wf * x0 + bf)
    c0 = i * u + f1 * c1 + f2 * c2
    h0 = o * math.tanh(c0)
    W = np.array([[wi], [wo], [wu], [wf]])
    b = np.array([bi, bo, bu, bf])
    U = np.array([[ui1, ui2], [uo1, uo2], [uu1, uu2], [0.0, u12], [0.0, 0.0]])
    f = wl.forest_from_parents([np.asarray([-1, 0, 0])])
    h, c = ob.forward_mixed(f.child_ptr, f.child_idx, np.array([[x0], [x1], [x2]]), [0, 0, 0], [dict(kind="nary", arity=2, W=W, U=U, b=b)])
    assert abs(h[0, 0] - h0) < 1e-15 and abs(c[0, 0] - c0) < 1e-15


def test_position_matters_and_swapping_children_swaps_blocks():
    rng = np.random.default_rng(9)
    D, H = 3, 2
    f = wl.forest_from_parents([np.asarray([-1, 0, 0, 1, 1, 2])])
    x = rng.standard_normal((f.n_nodes, D))
    W, _, b = wl.make_weights(rng, D, H, "normal", "random")
    U = rng.standard_normal((5 * H, 2 * H)) * 0.5
    cell = dict(kind="nary", arity=2, W=W, U=U, b=b)
    h, c = ob.forward_mixed(f.child_ptr, f.child_idx, x, np.zeros(6, dtype=int), [cell])
    # children listed in the other order
    idx = f.child_idx.copy()
    for v in range(f.n_nodes):
        a, e = f.child_ptr[v], f.child_ptr[v + 1]
        idx[a:e] = idx[a:e][::-1]
    hs, cs = ob.forward_mixed(f.child_ptr, idx, x, np.zeros(6, dtype=int), [cell])
    assert np.max(np.abs(hs[0] - h[0])) > 1e-3                   # position-dependent weights: the order matters
    # ... unless the blocks move with the children: column blocks swapped, forget row blocks swapped.  Node 2 has one
    # child, which the swap leaves in position 1, so the identity holds for the nodes whose child lists are full.
    Us = np.concatenate([U[:, H:], U[:, :H]], axis=1)
    Us = np.concatenate([Us[:3 * H], Us[4 * H:], Us[3 * H:4 * H]])
    f2 = wl.forest_from_parents([np.asarray([-1, 0, 0, 1, 1, 2, 2])])
    x2 = rng.standard_normal((7, D))
    h_a, c_a = ob.forward_mixed(f2.child_ptr, f2.child_idx, x2, np.zeros(7, dtype=int), [cell])
    idx2 = f2.child_idx.copy()
    for v in range(7):
        a, e = f2.child_ptr[v], f2.child_ptr[v + 1]
        idx2[a:e] = idx2[a:e][::-1]
    h_b, c_b = ob.forward_mixed(f2.child_ptr, idx2, x2, np.zeros(7, dtype=int), [dict(cell, U=Us)])
    assert np.max(np.abs(h_a - h_b)) < 1e-13 and np.max(np.abs(c_a - c_b)) < 1e-13


def test_mixed_forest_is_each_tree_alone_and_too_many_children_is_an_error():
    rng = np.random.default_rng(6)
    trees = wl._trees_capped(rng, 10, 3, 20, 2)
    f = wl.forest_from_parents(trees)
    D, H = 4, 3
    W0, U0, b0 = wl.make_weights(rng, D, H, "normal", "random")
    W1, _, b1 = wl.make_weights(rng, D, H, "normal", "random")
    cells = [dict(kind="childsum", W=W0, U=U0, b=b0), dict(kind="nary", arity=2, W=W1, U=rng.standard_normal((5 * H, 2 * H)) * 0.4, b=b1)]
    key = rng.integers(0, 2, size=f.n_nodes)
    x = rng.standard_normal((f.n_nodes, D))
    h, c = ob.forward_mixed(f.child_ptr, f.child_idx, x, key, cells)
    for t in range(f.n_trees):
        sub, nodes = wl.subforest(f, [t])
        hs, cs = ob.forward_mixed(sub.child_ptr, sub.child_idx, x[nodes], key[nodes], cells)
        assert np.array_equal(hs, h[nodes]) and np.array_equal(cs, c[nodes])
    star = wl.forest_from_parents([np.asarray([-1, 0, 0, 0])])
    try:
        ob.forward_mixed(star.child_ptr, star.child_idx, np.zeros((4, D)), [1, 0, 0, 0], cells)
        raise AssertionError("three children in a binary cell must be refused")
    except ValueError:
        pass
