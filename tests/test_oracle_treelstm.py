"""Pins for the CPU Tree-LSTM checker (oracle/treelstm.py).

Each pin is something the definition fixes without re-typing the checker:
a leaf is an LSTM cell with zero state; a single-child chain is an LSTM unrolled
(checked against torch's LSTMCell, a library routine with its own gate order);
a star over identical leaves has a closed form; a forest evaluates to the same
values as each tree alone, under any relabelling and any child order; degenerate
weights collapse the cell; a scalar two-child cell is worked out with math.exp.
"""
import math

import numpy as np
import pytest
import torch

from oracle import treelstm as ot
from paper_1904_07421_b200 import workloads as wl


def _sig(t):
    return 1.0 / (1.0 + math.exp(-t))


def _x(w):
    return w.x_full().astype(np.float64)


def test_leaf_is_zero_state_lstm_cell():
    w = wl.make_custom([[-1], [-1], [-1]], D=7, H=5, seed=1)
    h, c = ot.forward(w.forest.child_ptr, w.forest.child_idx, _x(w), w.W, w.U, w.b)
    H = w.H
    for v in range(3):
        x = _x(w)[v]
        for j in range(H):
            zi = sum(float(w.W[j, d]) * x[d] for d in range(w.D)) + float(w.b[j])
            zo = sum(float(w.W[H + j, d]) * x[d] for d in range(w.D)) + float(w.b[H + j])
            zu = sum(float(w.W[2 * H + j, d]) * x[d] for d in range(w.D)) + float(w.b[2 * H + j])
            cj = _sig(zi) * math.tanh(zu)
            assert abs(c[v, j] - cj) < 1e-14
            assert abs(h[v, j] - _sig(zo) * math.tanh(cj)) < 1e-14


def test_chain_equals_library_lstm_cell():
    """Node t's only child is node t+1: an LSTM run from the last node back to node 0."""
    T, D, H = 9, 6, 4
    w = wl.make_custom([[-1] + list(range(T - 1))], D=D, H=H, seed=2)
    h, c = ot.forward(w.forest.child_ptr, w.forest.child_idx, _x(w), w.W, w.U, w.b)

    cell = torch.nn.LSTMCell(D, H, bias=True, dtype=torch.float64)
    # torch orders its gates (input, forget, cell, output); ours are (i, o, u, f)
    blk = lambda M, g: torch.from_numpy(np.asarray(M[g * H:(g + 1) * H], dtype=np.float64))
    with torch.no_grad():
        cell.weight_ih.copy_(torch.cat([blk(w.W, 0), blk(w.W, 3), blk(w.W, 2), blk(w.W, 1)]))
        cell.weight_hh.copy_(torch.cat([blk(w.U, 0), blk(w.U, 3), blk(w.U, 2), blk(w.U, 1)]))
        cell.bias_ih.copy_(torch.cat([blk(w.b, 0), blk(w.b, 3), blk(w.b, 2), blk(w.b, 1)]))
        cell.bias_hh.zero_()
        hs = torch.zeros(1, H, dtype=torch.float64)
        cs = torch.zeros(1, H, dtype=torch.float64)
        x = torch.from_numpy(_x(w))
        for t in range(T - 1, -1, -1):
            hs, cs = cell(x[t:t + 1], (hs, cs))
            assert np.allclose(h[t], hs[0].numpy(), rtol=0, atol=1e-13)
            assert np.allclose(c[t], cs[0].numpy(), rtol=0, atol=1e-13)


def test_star_over_identical_leaves_closed_form():
    k, D, H = 6, 5, 3
    w = wl.make_custom([[-1] + [0] * k], D=D, H=H, seed=3)
    w.token[1:] = w.token[1]                      # identical leaves
    x = _x(w)
    h, c = ot.forward(w.forest.child_ptr, w.forest.child_idx, x, w.W, w.U, w.b)
    W, U, b = (a.astype(np.float64) for a in (w.W, w.U, w.b))
    z1 = W @ x[1] + b
    c_leaf = (1 / (1 + np.exp(-z1[0:H]))) * np.tanh(z1[2 * H:3 * H])
    h_leaf = (1 / (1 + np.exp(-z1[H:2 * H]))) * np.tanh(c_leaf)
    assert np.allclose(c[1:], c_leaf, atol=1e-14) and np.allclose(h[1:], h_leaf, atol=1e-14)
    z0 = W @ x[0] + b
    pre = z0[:3 * H] + U[:3 * H] @ (k * h_leaf)            # h~ = k * h_leaf
    f = 1 / (1 + np.exp(-(z0[3 * H:] + U[3 * H:] @ h_leaf)))  # same f for every child
    c_root = (1 / (1 + np.exp(-pre[0:H]))) * np.tanh(pre[2 * H:3 * H]) + k * f * c_leaf
    h_root = (1 / (1 + np.exp(-pre[H:2 * H]))) * np.tanh(c_root)
    assert np.allclose(c[0], c_root, atol=1e-13) and np.allclose(h[0], h_root, atol=1e-13)


def test_scalar_two_child_cell_by_hand():
    """D = H = 1, two different leaves; every number written out with math.exp."""
    f = wl.forest_from_parents([np.array([-1, 0, 0])])
    x = np.array([[0.5], [-1.25], [2.0]])
    W = np.array([[0.3], [-0.7], [1.1], [0.4]])      # i, o, u, f
    U = np.array([[-0.2], [0.9], [0.6], [-1.3]])
    b = np.array([0.05, -0.1, 0.2, 0.3])
    h, c = ot.forward(f.child_ptr, f.child_idx, x, W, U, b)

    def leaf(xv):
        cc = _sig(0.3 * xv + 0.05) * math.tanh(1.1 * xv + 0.2)
        return _sig(-0.7 * xv - 0.1) * math.tanh(cc), cc

    h1, c1 = leaf(-1.25)
    h2, c2 = leaf(2.0)
    hs = h1 + h2
    i = _sig(0.3 * 0.5 + 0.05 - 0.2 * hs)
    o = _sig(-0.7 * 0.5 - 0.1 + 0.9 * hs)
    u = math.tanh(1.1 * 0.5 + 0.2 + 0.6 * hs)
    f1 = _sig(0.4 * 0.5 + 0.3 - 1.3 * h1)
    f2 = _sig(0.4 * 0.5 + 0.3 - 1.3 * h2)
    c0 = i * u + f1 * c1 + f2 * c2
    h0 = o * math.tanh(c0)
    assert abs(c[0, 0] - c0) < 1e-15 and abs(h[0, 0] - h0) < 1e-15
    assert abs(h[1, 0] - h1) < 1e-15 and abs(c[2, 0] - c2) < 1e-15


def test_batched_equals_unbatched_and_relabelled():
    w = wl.make_workload(1, n_trees=12)
    f = w.forest
    x = _x(w)
    h, c = ot.forward(f.child_ptr, f.child_idx, x, w.W, w.U, w.b)
    assert not np.isnan(h).any()
    # each tree alone
    for t in range(f.n_trees):
        sub, nodes = wl.subforest(f, [t])
        hs, cs = ot.forward(sub.child_ptr, sub.child_idx, x[nodes], w.W, w.U, w.b)
        assert np.max(np.abs(hs - h[nodes])) < 1e-12 and np.max(np.abs(cs - c[nodes])) < 1e-12
    # only some roots evaluated: untouched trees stay NaN, touched ones agree
    h2, c2 = ot.forward(f.child_ptr, f.child_idx, x, w.W, w.U, w.b, roots=f.roots[:3])
    a, b_ = int(f.tree_ptr[0]), int(f.tree_ptr[3])
    assert np.array_equal(h2[a:b_], h[a:b_]) and np.isnan(h2[b_:]).all()
    # random relabelling + shuffled child lists
    rng = np.random.default_rng(5)
    g, new_id = wl.relabel(f, rng, shuffle_children=True)
    xr = np.empty_like(x)
    xr[new_id] = x
    hr, cr = ot.forward(g.child_ptr, g.child_idx, xr, w.W, w.U, w.b)
    assert np.max(np.abs(hr[new_id] - h)) < 1e-12 and np.max(np.abs(cr[new_id] - c)) < 1e-12


def test_degenerate_weights():
    w = wl.make_workload(1, n_trees=6)
    f = w.forest
    x = _x(w)
    Z = lambda a: np.zeros_like(a)
    h, c = ot.forward(f.child_ptr, f.child_idx, x, Z(w.W), Z(w.U), Z(w.b))
    assert np.all(h == 0) and np.all(c == 0)          # u = tanh(0) = 0 everywhere
    # U = 0: gates depend on x only and c_j = i*u + sigmoid(z_f) * sum_k c_k
    rng = np.random.default_rng(9)
    b = rng.uniform(-0.5, 0.5, size=w.b.shape)
    h, c = ot.forward(f.child_ptr, f.child_idx, x, w.W, Z(w.U), b)
    z = x @ w.W.astype(np.float64).T + b
    H = w.H
    sg = lambda t: 1 / (1 + np.exp(-t))
    parent = wl.parent_array(f)
    csum = np.zeros_like(c)
    for v in range(f.n_nodes):
        if parent[v] >= 0:
            csum[parent[v]] += c[v]
    expect_c = sg(z[:, :H]) * np.tanh(z[:, 2 * H:3 * H]) + sg(z[:, 3 * H:]) * csum
    assert np.max(np.abs(expect_c - c)) < 1e-12
    assert np.max(np.abs(sg(z[:, H:2 * H]) * np.tanh(expect_c) - h)) < 1e-12


def test_bf16_rounding_matches_library_conversion():
    rng = np.random.default_rng(11)
    a = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, size=4096),
                        np.array([0.0, 1.0, 1.00390625, 1.01171875, -3.0e38, 1e-40])]).astype(np.float32)
    lib = torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ot.bf16_round(a), lib)
    assert np.array_equal(wl.round_to_bf16(a).astype(np.float64), lib)


def test_quantised_mode_stays_close_to_plain():
    w = wl.make_workload(2, n_trees=16)
    f = w.forest
    x = _x(w)
    h, c = ot.forward(f.child_ptr, f.child_idx, x, w.W, w.U, w.b)
    hq, cq = ot.forward(f.child_ptr, f.child_idx, x, w.W, w.U, w.b, quantize="bf16")
    err = max(np.max(np.abs(h - hq)), np.max(np.abs(c - cq)))
    assert 0 < err < 3e-2


def test_edge_rounding_mode_equals_sum_rounding_where_the_sum_needs_no_rounding():
    """bf16_edges rounds h_k and leaves the sum of the rounded rows alone; bf16 rounds the sum.  Where every node
    has at most one child the sum IS the rounded row, and twice a bfloat16 value is a bfloat16 value, so chains
    and pairs of identical leaves must agree exactly; three different children must not (but stay close)."""
    rng = np.random.default_rng(23)
    H, D = 12, 9
    W = rng.uniform(-0.5, 0.5, (4 * H, D))
    U = rng.uniform(-0.5, 0.5, (4 * H, H))
    b = rng.uniform(-0.5, 0.5, 4 * H)
    chain = wl.forest_from_parents([np.array([-1] + list(range(9)))])
    x = rng.standard_normal((chain.n_nodes, D))
    a = ot.forward(chain.child_ptr, chain.child_idx, x, W, U, b, quantize="bf16")
    e = ot.forward(chain.child_ptr, chain.child_idx, x, W, U, b, quantize="bf16_edges")
    assert np.array_equal(a[0], e[0]) and np.array_equal(a[1], e[1])
    twins = wl.forest_from_parents([np.array([-1, 0, 0])])
    x = rng.standard_normal((3, D))
    x[2] = x[1]
    a = ot.forward(twins.child_ptr, twins.child_idx, x, W, U, b, quantize="bf16")
    e = ot.forward(twins.child_ptr, twins.child_idx, x, W, U, b, quantize="bf16_edges")
    assert np.array_equal(a[0], e[0]) and np.array_equal(a[1], e[1])
    three = wl.forest_from_parents([np.array([-1, 0, 0, 0])])
    x = rng.standard_normal((4, D))
    a = ot.forward(three.child_ptr, three.child_idx, x, W, U, b, quantize="bf16")
    e = ot.forward(three.child_ptr, three.child_idx, x, W, U, b, quantize="bf16_edges")
    p = ot.forward(three.child_ptr, three.child_idx, x, W, U, b)
    assert np.array_equal(a[0][1:], e[0][1:])                      # the leaves do not depend on the mode
    assert 0 < np.max(np.abs(a[0][0] - e[0][0])) < 2e-2
    assert np.max(np.abs(p[0] - e[0])) < 3e-2 and np.max(np.abs(p[1] - e[1])) < 3e-2


def test_x_of_callback_equals_array():
    w = wl.make_workload(1, n_trees=4)
    f = w.forest
    h, c = ot.forward(f.child_ptr, f.child_idx, _x(w), w.W, w.U, w.b)
    h2, c2 = ot.forward(f.child_ptr, f.child_idx, None, w.W, w.U, w.b, x_of=lambda v: w.table[w.token[v]])
    assert np.array_equal(h, h2) and np.array_equal(c, c2)


# ---- where the bf16-matched modes round -----------------------------------------------------------------
# A scalar cell (D = H = 1) over one root with two different leaves, worked with math.exp.  Every rounded value is
# typed here as a literal; that a literal is THE bfloat16 neighbour of the value it stands for is checked from the
# format's definition (8 significant bits, within half a unit in the last place), not with the checker's routine.
def _is_bf16(v):
    m, _ = math.frexp(v)
    return float(m * 256.0).is_integer()


def _is_nearest_bf16(v, lit):
    _, e = math.frexp(v)                       # |v| in [2^(e-1), 2^e): one unit in the last place is 2^(e-8)
    half = 2.0 ** (e - 9)
    m, _ = math.frexp(lit)
    even = int(abs(m) * 256.0) % 2 == 0        # a value half-way between two neighbours goes to the even one
    return _is_bf16(lit) and (abs(v - lit) < half or (abs(v - lit) == half and even))


_RX = [0.5029296875, 0.28271484375, 1.0341796875]                      # x of root, leaf 1, leaf 2
_RW = [0.301513671875, -0.70263671875, 1.10498046875, 0.40087890625]  # i, o, u, f
_RU = [-0.200439453125, 0.90185546875, 0.60107421875, -1.3076171875]
_RB = [0.05, -0.1, 0.2, 0.3]                                          # the bias is never rounded
_RXQ = [0.50390625, 0.283203125, 1.03125]
_RWQ = [0.30078125, -0.703125, 1.1015625, 0.400390625]
_RUQ = [-0.2001953125, 0.90234375, 0.6015625, -1.3046875]
# bfloat16 neighbours of the leaves' h computed from the rounded inputs (h_1 = 0.104938..., h_2 = 0.143876...), of their
# sum (0.248814...), and of the sum of the two rounded rows (0.24853515625, half-way between two neighbours)
_RH1Q, _RH2Q, _RHSUMQ, _RHROWSQ = 0.10498046875, 0.1435546875, 0.2490234375, 0.248046875


def _rounding_chain(mode, drop=None):
    """(h_root, c_root, h_1, h_2) of the scalar cell, with the roundings of `mode` minus the one named by `drop`."""
    r = lambda name, raw, rounded: raw if (mode is None or drop == name) else rounded
    x = [r("x", a, b) for a, b in zip(_RX, _RXQ)]
    W = [r("W", a, b) for a, b in zip(_RW, _RWQ)]
    U = [r("U", a, b) for a, b in zip(_RU, _RUQ)]

    def leaf(xv):
        cc = _sig(W[0] * xv + _RB[0]) * math.tanh(W[2] * xv + _RB[2])
        return _sig(W[1] * xv + _RB[1]) * math.tanh(cc), cc

    (h1, c1), (h2, c2) = leaf(x[1]), leaf(x[2])
    if mode is not None and drop is None:
        assert _is_nearest_bf16(h1, _RH1Q) and _is_nearest_bf16(h2, _RH2Q) and _is_nearest_bf16(h1 + h2, _RHSUMQ)
        assert _is_nearest_bf16(_RH1Q + _RH2Q, _RHROWSQ) and _RH1Q + _RH2Q != _RHROWSQ
    h1q, h2q = r("h_k", h1, _RH1Q), r("h_k", h2, _RH2Q)
    if mode == "bf16":
        hs = r("h_sum", h1 + h2, _RHSUMQ)        # the child sum of the exact rows, rounded once
    elif mode == "bf16_edges":
        hs = h1q + h2q                            # the rounded rows, added exactly
    elif mode == "bf16_rows":
        hs = r("h_sum", h1q + h2q, _RHROWSQ)      # the rounded rows, added exactly, the sum rounded again
    else:
        hs = h1 + h2
    i = _sig(W[0] * x[0] + _RB[0] + U[0] * hs)
    o = _sig(W[1] * x[0] + _RB[1] + U[1] * hs)
    u = math.tanh(W[2] * x[0] + _RB[2] + U[2] * hs)
    f1 = _sig(W[3] * x[0] + _RB[3] + U[3] * h1q)
    f2 = _sig(W[3] * x[0] + _RB[3] + U[3] * h2q)
    c0 = i * u + f1 * c1 + f2 * c2                # c_k is state: never rounded
    return o * math.tanh(c0), c0, h1, h2


@pytest.mark.parametrize("mode", [None, "bf16", "bf16_edges", "bf16_rows"])
def test_rounding_points_of_the_matched_modes_by_hand(mode):
    for raw, lit in zip(_RX + _RW + _RU, _RXQ + _RWQ + _RUQ):
        assert raw != lit and _is_nearest_bf16(raw, lit)
    f = wl.forest_from_parents([np.array([-1, 0, 0])])
    h, c = ot.forward(f.child_ptr, f.child_idx, np.array(_RX).reshape(3, 1), np.array(_RW).reshape(4, 1),
                      np.array(_RU).reshape(4, 1), np.array(_RB), quantize=mode)
    h0, c0, h1, h2 = _rounding_chain(mode)
    assert abs(h[0, 0] - h0) < 1e-15 and abs(c[0, 0] - c0) < 1e-15
    assert abs(h[1, 0] - h1) < 1e-15 and abs(h[2, 0] - h2) < 1e-15
    if mode is None:
        return
    # a checker that forgot any one of the roundings would land on one of these chains instead: each is far away
    points = ["x", "W", "U", "h_k"] + (["h_sum"] if mode != "bf16_edges" else [])
    for drop in points:
        hd, cd, _, _ = _rounding_chain(mode, drop)
        assert max(abs(hd - h[0, 0]), abs(cd - c[0, 0])) > 2e-6, drop
    # and the two modes differ from each other and from the plain evaluation
    for other in {"bf16", "bf16_edges", "bf16_rows"} - {mode}:
        assert abs(_rounding_chain(other)[0] - h0) > 1e-6, other
    assert abs(_rounding_chain(None)[0] - h0) > 1e-4
