"""Child-Sum Tree-LSTM forward, one node at a time in fp64.  TEST INFRASTRUCTURE ONLY.

The paper batches the cells of a Tree-LSTM (Section 3 cites the Child-Sum
Tree-LSTM and counts 33 operators per cell, 4 of which depend on the number of
children) and states that batching leaves every result unchanged (Section 1,
the isomorphism guarantee).  So the reference result is simply the unbatched
cell applied node by node, children before parents.  For node j with input x_j
and children C(j), with gate row blocks (i, o, u, f) of W [4H, D], U [4H, H],
b [4H]:

    h~_j  = sum_{k in C(j)} h_k                       (zero vector for a leaf)
    i_j   = sigmoid(W_i x_j + U_i h~_j + b_i)
    o_j   = sigmoid(W_o x_j + U_o h~_j + b_o)
    u_j   = tanh   (W_u x_j + U_u h~_j + b_u)
    f_jk  = sigmoid(W_f x_j + U_f h_k  + b_f)         one per child k
    c_j   = i_j * u_j + sum_{k in C(j)} f_jk * c_k
    h_j   = o_j * tanh(c_j)

Readings where the paper is silent: the gate order and weight orientation above;
the forget gate of child k uses the parent's input x_j and the child's own h_k;
children are summed in CSR order.

``quantize="bf16"`` rounds exactly those values to bfloat16 that a bf16 GEMM path
must round (x, W, U and the GEMM operands h~_j and h_k) and keeps everything else
in fp64, so that rounding can be told apart from a mistake.
``quantize="bf16_edges"`` is the same for an evaluation that takes the child sum
behind the product, U_iou h~_j = sum_k U_iou h_k: the only recurrent GEMM operand is
then h_k, so each h_k is rounded and the sum of the rounded rows is not rounded again.
``quantize="bf16_rows"`` is the evaluation that keeps only a bf16 copy of every h_k for
the recurrence: the child sum is taken over the rounded rows and, being a GEMM operand
itself, is rounded once more, h~_j = bf16(sum_k bf16(h_k)).
The paper fixes no precision; all three are bf16-GEMM evaluations of the same cell.

Nothing here is shared with the CUDA path.  Pins: tests/test_oracle_treelstm.py.
"""
from __future__ import annotations

import numpy as np


def sigmoid(t):
    return 1.0 / (1.0 + np.exp(-t))


def bf16_round(a):
    """Nearest bfloat16 (ties to even) of fp64/fp32 values, returned as fp64."""
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    bits = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return bits.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))


def _postorder(child_ptr, child_idx, roots):
    """Nodes reachable from ``roots``, every child before its parent (explicit stack)."""
    order = []
    stack = [(int(r), False) for r in reversed(list(roots))]
    while stack:
        v, expanded = stack.pop()
        if expanded:
            order.append(v)
            continue
        stack.append((v, True))
        for e in range(int(child_ptr[v + 1]) - 1, int(child_ptr[v]) - 1, -1):
            stack.append((int(child_idx[e]), False))
    return order


def find_roots(child_ptr, child_idx, n_nodes):
    has_parent = np.zeros(n_nodes, dtype=bool)
    has_parent[np.asarray(child_idx, dtype=np.int64)] = True
    return np.nonzero(~has_parent)[0]


def forward(child_ptr, child_idx, x, W, U, b, roots=None, quantize=None, x_of=None):
    """Evaluate the trees under ``roots`` (default: every tree).

    x      : [n_nodes, D] array, or None when ``x_of(v)`` supplies the row of node v.
    Returns (h, c) fp64 [n_nodes, H]; rows of nodes that were not evaluated are NaN.
    """
    child_ptr = np.asarray(child_ptr, dtype=np.int64)
    child_idx = np.asarray(child_idx, dtype=np.int64)
    n = child_ptr.shape[0] - 1
    W = np.asarray(W, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    H = U.shape[1]
    assert W.shape[0] == 4 * H and U.shape[0] == 4 * H and b.shape[0] == 4 * H
    q = (lambda a: a) if quantize is None else bf16_round
    if quantize not in (None, "bf16", "bf16_edges", "bf16_rows"):
        raise ValueError(quantize)
    W = q(W)
    U = q(U)
    U_i, U_o, U_u, U_f = U[0:H], U[H:2 * H], U[2 * H:3 * H], U[3 * H:4 * H]
    if roots is None:
        roots = find_roots(child_ptr, child_idx, n)

    h = np.full((n, H), np.nan, dtype=np.float64)
    c = np.full((n, H), np.nan, dtype=np.float64)
    for j in _postorder(child_ptr, child_idx, roots):
        xj = np.asarray(x_of(j) if x is None else x[j], dtype=np.float64)
        xj = q(xj)
        kids = child_idx[child_ptr[j]:child_ptr[j + 1]]
        h_sum = np.zeros(H, dtype=np.float64)
        for k in kids:
            h_sum = h_sum + h[k]
        z = W @ xj + b
        z_i, z_o, z_u, z_f = z[0:H], z[H:2 * H], z[2 * H:3 * H], z[3 * H:4 * H]
        if quantize in ("bf16_edges", "bf16_rows"):
            hs = np.zeros(H, dtype=np.float64)
            for k in kids:
                hs = hs + q(h[k])
            if quantize == "bf16_rows":
                hs = q(hs)
        else:
            hs = q(h_sum)
        i = sigmoid(z_i + U_i @ hs)
        o = sigmoid(z_o + U_o @ hs)
        u = np.tanh(z_u + U_u @ hs)
        cj = i * u
        for k in kids:
            f_k = sigmoid(z_f + U_f @ q(h[k]))
            cj = cj + f_k * c[k]
        c[j] = cj
        h[j] = o * np.tanh(cj)
    return h, c
