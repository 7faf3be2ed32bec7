"""Pins for the reverse-mode checker (oracle/treelstm_backward.py): finite differences, a library cell's autograd,
and forest = trees one by one."""
import numpy as np
import torch

from oracle import treelstm as ot
from oracle import treelstm_backward as ob
from paper_1904_07421_b200 import workloads as wl


def _case(parents, D, H, seed):
    w = wl.make_custom(parents, D=D, H=H, seed=seed, bias="random")
    f = w.forest
    rng = np.random.default_rng(seed + 1)
    x = w.x_full().astype(np.float64)
    gh = rng.standard_normal((f.n_nodes, H))
    gc = rng.standard_normal((f.n_nodes, H)) * 0.5
    return f, x, w.W.astype(np.float64), w.U.astype(np.float64), w.b.astype(np.float64), gh, gc


def _loss(f, x, W, U, b, gh, gc):
    h, c = ot.forward(f.child_ptr, f.child_idx, x, W, U, b)
    return float(np.sum(gh * h) + np.sum(gc * c))


def test_central_differences_in_every_block():
    """Trees with 0, 1, 2 and 3 children per node, every node in the loss through h and c."""
    f, x, W, U, b, gh, gc = _case([[-1, 0, 0, 1, 1, 1, 2], [-1, 0, 1], [-1]], D=3, H=2, seed=5)
    dW, dU, db, dx = ob.backward(f.child_ptr, f.child_idx, x, W, U, b, gh, gc)
    eps = 1e-6
    for name, arr, grad in (("W", W, dW), ("U", U, dU), ("b", b, db), ("x", x, dx)):
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = arr[idx]
            arr[idx] = keep + eps
            up = _loss(f, x, W, U, b, gh, gc)
            arr[idx] = keep - eps
            down = _loss(f, x, W, U, b, gh, gc)
            arr[idx] = keep
            assert abs((up - down) / (2 * eps) - grad[idx]) < 2e-8, (name, idx)


def test_chain_against_library_lstm_autograd():
    T, D, H = 7, 5, 4
    f, x, W, U, b, gh, gc = _case([[-1] + list(range(T - 1))], D=D, H=H, seed=8)
    dW, dU, db, dx = ob.backward(f.child_ptr, f.child_idx, x, W, U, b, gh, gc)
    cell = torch.nn.LSTMCell(D, H, bias=True, dtype=torch.float64)
    order = [0, 3, 2, 1]                      # torch's gate order (input, forget, cell, output) in ours (i, o, u, f)
    blk = lambda M: torch.cat([torch.from_numpy(M[g * H:(g + 1) * H]) for g in order])
    with torch.no_grad():
        cell.weight_ih.copy_(blk(W))
        cell.weight_hh.copy_(blk(U))
        cell.bias_ih.copy_(blk(b))
        cell.bias_hh.zero_()
    xt = torch.from_numpy(x).requires_grad_(True)
    hs = torch.zeros(1, H, dtype=torch.float64)
    cs = torch.zeros(1, H, dtype=torch.float64)
    loss = 0.0
    for t in range(T - 1, -1, -1):            # node t's only child is node t + 1
        hs, cs = cell(xt[t:t + 1], (hs, cs))
        loss = loss + (torch.from_numpy(gh[t]) * hs[0]).sum() + (torch.from_numpy(gc[t]) * cs[0]).sum()
    loss.backward()
    back = lambda G: np.concatenate([G[order.index(g) * H:(order.index(g) + 1) * H] for g in range(4)])
    assert np.allclose(back(cell.weight_ih.grad.numpy()), dW, rtol=0, atol=1e-12)
    assert np.allclose(back(cell.weight_hh.grad.numpy()), dU, rtol=0, atol=1e-12)
    assert np.allclose(back(cell.bias_ih.grad.numpy()), db, rtol=0, atol=1e-12)
    assert np.allclose(xt.grad.numpy(), dx, rtol=0, atol=1e-12)


def test_forest_equals_its_trees_and_relabelling():
    w = wl.make_workload(1, n_trees=5, bias="random")
    f = w.forest
    rng = np.random.default_rng(2)
    H = w.H
    x = w.x_full().astype(np.float64)
    gh = np.zeros((f.n_nodes, H))
    gh[f.roots] = rng.standard_normal((f.n_trees, H))        # the loss looks at the roots only
    dW, dU, db, dx = ob.backward(f.child_ptr, f.child_idx, x, w.W, w.U, w.b, gh)
    sW, sU, sb = np.zeros_like(dW), np.zeros_like(dU), np.zeros_like(db)
    for t in range(f.n_trees):
        sub, nodes = wl.subforest(f, [t])
        tW, tU, tb, tx = ob.backward(sub.child_ptr, sub.child_idx, x[nodes], w.W, w.U, w.b, gh[nodes])
        sW += tW; sU += tU; sb += tb
        assert np.max(np.abs(tx - dx[nodes])) < 1e-12
    assert np.max(np.abs(sW - dW)) < 1e-10 and np.max(np.abs(sU - dU)) < 1e-10 and np.max(np.abs(sb - db)) < 1e-10
    g, new_id = wl.relabel(f, np.random.default_rng(6))
    xr, ghr = np.empty_like(x), np.empty_like(gh)
    xr[new_id], ghr[new_id] = x, gh
    rW, rU, rb, rx = ob.backward(g.child_ptr, g.child_idx, xr, w.W, w.U, w.b, ghr)
    assert np.max(np.abs(rW - dW)) < 1e-10 and np.max(np.abs(rU - dU)) < 1e-10 and np.max(np.abs(rx[new_id] - dx)) < 1e-12
