"""The depth table for nodes of several kinds, and a forest whose cells are of two kinds.  TEST INFRASTRUCTURE ONLY.

Section 4.2 of the paper files every recorded node under a key made of its type, its settings, the layout of its
arguments and its result index, together with its depth; nodes that share key and depth share a slot and run as one
batched launch (Section 4.3), the slots in depth order.  Here a node carries one integer `key` that stands for
(type, settings, layout): nodes with equal key are batchable with each other, nodes with different keys are not.

    plan(...)            the table: node ids ordered by (depth, key, id) and the slot boundaries;
    forward_mixed(...)   h and c of every node of a forest in which `key[v]` selects node v's cell from a list:
                         the Child-Sum cell of oracle/treelstm.py, or the N-ary Tree-LSTM cell of the same cited
                         model, which keeps one recurrent matrix per child POSITION:

        i   = sig (W_i x + sum_l U_i^l  h_l + b_i)         o, u alike (u through tanh)
        f_k = sig (W_f x + sum_l U_f^kl h_l + b_f)          k = 1 .. arity
        c   = i * u + sum_k f_k * c_k                       h = o * tanh(c)

    A missing child (fewer children than the arity) contributes h_l = c_l = 0; more children than the arity is an
    error.  Weight layout: W [4H, D] and b [4H] in row blocks (i, o, u, f); U [(3 + arity) H, arity H] in row blocks
    (i, o, u, f_1 .. f_arity) and column blocks l = 1 .. arity.

Readings where the paper is silent: slots are ordered by (depth, key) and ids ascend inside a slot; depth is the height
above the leaves (as in oracle/schedule.py), whatever the kinds of the nodes below.

Nothing here is shared with the CUDA path.  Pins: tests/test_oracle_batcher.py.
"""
from __future__ import annotations

import numpy as np

from oracle.schedule import schedule
from oracle.treelstm import _postorder, find_roots, sigmoid


def plan(child_ptr, child_idx, key):
    """(perm, slot_ptr, slot_depth, slot_key, depth) of the forest's nodes filed by (depth, key)."""
    key = np.asarray(key, dtype=np.int64)
    n = key.shape[0]
    depth = schedule(child_ptr, child_idx, n)[0].astype(np.int64) if n else np.zeros(0, dtype=np.int64)
    filed = {}
    for v in range(n):                                   # one node at a time into its slot
        filed.setdefault((int(depth[v]), int(key[v])), []).append(v)
    perm, slot_ptr, slot_depth, slot_key = [], [0], [], []
    for (d, k) in sorted(filed):
        perm.extend(filed[(d, k)])
        slot_ptr.append(len(perm))
        slot_depth.append(d)
        slot_key.append(k)
    as_i = lambda a: np.asarray(a, dtype=np.int64)
    return as_i(perm), as_i(slot_ptr), as_i(slot_depth), as_i(slot_key), depth


def childsum_cell(x, hs, cs, W, U, b):
    """One Child-Sum cell: hs, cs are the lists of the children's states."""
    H = U.shape[1]
    h_sum = np.zeros(H)
    for hk in hs:
        h_sum = h_sum + hk
    z = W @ x + b
    i = sigmoid(z[0:H] + U[0:H] @ h_sum)
    o = sigmoid(z[H:2 * H] + U[H:2 * H] @ h_sum)
    u = np.tanh(z[2 * H:3 * H] + U[2 * H:3 * H] @ h_sum)
    c = i * u
    for hk, ck in zip(hs, cs):
        c = c + sigmoid(z[3 * H:] + U[3 * H:] @ hk) * ck
    return o * np.tanh(c), c


def nary_cell(x, hs, cs, W, U, b, arity):
    """One N-ary cell: child l's state multiplies column block l of U."""
    H = U.shape[1] // arity
    if len(hs) > arity:
        raise ValueError(f"node with {len(hs)} children in a cell of arity {arity}")
    z = W @ x + b
    rec = np.zeros((3 + arity) * H)
    for l, hl in enumerate(hs):
        rec = rec + U[:, l * H:(l + 1) * H] @ hl
    i = sigmoid(z[0:H] + rec[0:H])
    o = sigmoid(z[H:2 * H] + rec[H:2 * H])
    u = np.tanh(z[2 * H:3 * H] + rec[2 * H:3 * H])
    c = i * u
    for k, ck in enumerate(cs):
        c = c + sigmoid(z[3 * H:] + rec[(3 + k) * H:(4 + k) * H]) * ck
    return o * np.tanh(c), c


def forward_mixed(child_ptr, child_idx, x, key, cells):
    """h, c [n, H] in fp64.  cells[k] = dict(kind="childsum" | "nary", W=, U=, b=, arity= (nary only))."""
    child_ptr = np.asarray(child_ptr, dtype=np.int64)
    child_idx = np.asarray(child_idx, dtype=np.int64)
    key = np.asarray(key, dtype=np.int64)
    n = child_ptr.shape[0] - 1
    x = np.asarray(x, dtype=np.float64)
    cells = [dict(c, W=np.asarray(c["W"], dtype=np.float64), U=np.asarray(c["U"], dtype=np.float64),
                  b=np.asarray(c["b"], dtype=np.float64)) for c in cells]
    H = cells[0]["W"].shape[0] // 4 if cells else 0
    h = np.zeros((n, H))
    c = np.zeros((n, H))
    for j in _postorder(child_ptr, child_idx, find_roots(child_ptr, child_idx, n)):
        kids = child_idx[child_ptr[j]:child_ptr[j + 1]]
        cell = cells[int(key[j])]
        hs, cs = [h[k] for k in kids], [c[k] for k in kids]
        if cell["kind"] == "childsum":
            h[j], c[j] = childsum_cell(x[j], hs, cs, cell["W"], cell["U"], cell["b"])
        elif cell["kind"] == "nary":
            h[j], c[j] = nary_cell(x[j], hs, cs, cell["W"], cell["U"], cell["b"], int(cell["arity"]))
        else:
            raise ValueError(cell["kind"])
    return h, c
