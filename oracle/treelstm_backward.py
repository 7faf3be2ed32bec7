"""Reverse-mode derivative of the Child-Sum Tree-LSTM forward, one node at a time in fp64.  TEST INFRASTRUCTURE ONLY.

The paper's training loop (the listing of Section 4.3) calls backward() inside the batching scope, and its speed
table (Section 5) reports training next to inference: the backward pass runs over the same depth table, levels in
DESCENDING order, because a node's gradient is complete once all of its parents (here: its one parent) are done.
This file is the plain definition of that pass for the cell of oracle/treelstm.py, written out per node:

    given dL/dh_j and dL/dc_j (what the loss and the parent contributed), with t = tanh(c_j):
        dc    = dL/dc_j + dL/dh_j * o * (1 - t^2)           do = dL/dh_j * t
        di    = dc * u        du = dc * i                    df_k = dc * c_k        dL/dc_k += dc * f_k
        dz_i  = di i (1 - i)  dz_o = do o (1 - o)  dz_u = du (1 - u^2)  dz_fk = df_k f_k (1 - f_k)
        dW   += [dz_i; dz_o; dz_u; sum_k dz_fk] x_j^T        db += [dz_i; dz_o; dz_u; sum_k dz_fk]
        dU_iou += [dz_i; dz_o; dz_u] h~_j^T                  dU_f += sum_k dz_fk h_k^T
        dL/dx_j = W^T [dz_i; dz_o; dz_u; sum_k dz_fk]
        dL/dh_k += U_iou^T [dz_i; dz_o; dz_u] + U_f^T dz_fk  for every child k

Nothing here is shared with the CUDA path (which has no backward pass yet).  Pins: tests/test_oracle_backward.py
(central differences of a scalar loss in every parameter block and in x; a library LSTM cell's autograd on chains;
a forest equals its trees one by one).
"""
from __future__ import annotations

import numpy as np

from oracle.treelstm import _postorder, find_roots, forward, sigmoid


def backward(child_ptr, child_idx, x, W, U, b, grad_h, grad_c=None):
    """Gradients of L = sum_v <grad_h[v], h_v> + <grad_c[v], c_v> (rows of nodes that do not enter the loss are zero).

    Returns (dW [4H, D], dU [4H, H], db [4H], dx [n, D]) in fp64.
    """
    child_ptr = np.asarray(child_ptr, dtype=np.int64)
    child_idx = np.asarray(child_idx, dtype=np.int64)
    n = child_ptr.shape[0] - 1
    x = np.asarray(x, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    H = U.shape[1]
    h, c = forward(child_ptr, child_idx, x, W, U, b)
    dh = np.array(grad_h, dtype=np.float64, copy=True)
    dc = np.zeros_like(dh) if grad_c is None else np.array(grad_c, dtype=np.float64, copy=True)
    dW, dU, db, dx = np.zeros_like(W), np.zeros_like(U), np.zeros_like(b), np.zeros_like(x)
    U_iou, U_f = U[:3 * H], U[3 * H:]
    order = _postorder(child_ptr, child_idx, find_roots(child_ptr, child_idx, n))
    for j in reversed(order):                       # every parent before its children
        kids = child_idx[child_ptr[j]:child_ptr[j + 1]]
        h_sum = np.zeros(H)
        for k in kids:
            h_sum = h_sum + h[k]
        z = W @ x[j] + b
        i = sigmoid(z[0:H] + U[0:H] @ h_sum)
        o = sigmoid(z[H:2 * H] + U[H:2 * H] @ h_sum)
        u = np.tanh(z[2 * H:3 * H] + U[2 * H:3 * H] @ h_sum)
        t = np.tanh(c[j])
        dcj = dc[j] + dh[j] * o * (1.0 - t * t)
        dz_i = dcj * u * i * (1.0 - i)
        dz_o = dh[j] * t * o * (1.0 - o)
        dz_u = dcj * i * (1.0 - u * u)
        dz_iou = np.concatenate([dz_i, dz_o, dz_u])
        dz_f_sum = np.zeros(H)
        dh_sum = U_iou.T @ dz_iou                   # what every child receives through the child sum
        for k in kids:
            f_k = sigmoid(z[3 * H:] + U_f @ h[k])
            dz_fk = dcj * c[k] * f_k * (1.0 - f_k)
            dc[k] = dc[k] + dcj * f_k
            dh[k] = dh[k] + dh_sum + U_f.T @ dz_fk
            dU[3 * H:] += np.outer(dz_fk, h[k])
            dz_f_sum = dz_f_sum + dz_fk
        dz = np.concatenate([dz_iou, dz_f_sum])
        dW += np.outer(dz, x[j])
        db += dz
        dU[:3 * H] += np.outer(dz_iou, h_sum)
        dx[j] = W.T @ dz
    return dW, dU, db, dx
