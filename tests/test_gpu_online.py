"""Requests arriving one after the other (jdb_online_*): every request's result is what the one-call host entry gives
for it, bit for bit, whatever the order of the waits, and an error stays with the request that caused it."""
import numpy as np
import pytest
import torch

from oracle import treelstm as ot
from paper_1904_07421_b200 import jdb
from paper_1904_07421_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _request(w, pin=True):
    f = w.forest
    dt = torch.bfloat16 if w.precision == "bf16" else torch.float32
    mk = lambda t: t.pin_memory() if pin else t
    cp, ci = mk(torch.from_numpy(f.child_ptr.astype(np.int32))), mk(torch.from_numpy(f.child_idx.astype(np.int32)))
    x = mk(torch.from_numpy(w.x_full()).to(dt).contiguous())
    h = mk(torch.full((f.n_nodes, w.H), float("nan"), dtype=torch.float32))
    c = mk(torch.full((f.n_nodes, w.H), float("nan"), dtype=torch.float32))
    return cp, ci, x, h, c


def _stream_of_requests(index, sizes, seed):
    """Forests of one workload shape and one set of weights, with different tree counts (a stream of requests)."""
    base = wl.make_workload(index, n_trees=4, bias="random")
    out = []
    for k, t in enumerate(sizes):
        wk = wl.make_workload(index, n_trees=t, seed=seed + k, bias="random")
        out.append(wl.Workload(wk.name, wk.index, wk.forest, wk.D, wk.H, wk.precision, base.table,
                               (wk.token % base.table.shape[0]).astype(np.int32), base.W, base.U, base.b))
    return base, out


@pytest.mark.parametrize("index,slots", [(2, 3), (1, 2), (3, 2)])
def test_every_request_equals_the_one_call_entry(index, slots):
    """bf16 cooperative loop, fp32, and bf16 per-level launches (which synchronise for their level count); twelve
    requests of 3 to 90 trees through 2 or 3 slots, waited for in a shuffled order."""
    sizes = [5, 90, 3, 40, 17, 64, 8, 33, 21, 70, 11, 50] if index != 3 else [4, 30, 9, 16, 22, 6]
    base, reqs = _stream_of_requests(index, sizes, seed=100 * index)
    precision = jdb.BF16 if base.precision == "bf16" else jdb.FP32
    packed = jdb.jdb_pack_weights(*(torch.from_numpy(a).to(DEV) for a in (base.W, base.U, base.b)), precision)
    x_dtype = precision
    max_n = max(r.forest.n_nodes for r in reqs)
    max_e = max(r.forest.n_edges for r in reqs)
    on = jdb.Online(slots, max_n, max_e, packed, base.D, base.H, precision, x_dtype, DEV)
    bufs = [_request(r) for r in reqs]
    tickets = [on.submit(*b) for b in bufs]
    assert tickets == list(range(len(reqs)))
    order = np.random.default_rng(index).permutation(len(reqs))
    levels = {}
    for k in order:
        levels[k] = on.wait(tickets[k])
    on.close()
    ws = jdb.forward_host_workspace(max_n, max_e, base.D, base.H, precision, x_dtype, DEV)
    for k, (r, b) in enumerate(zip(reqs, bufs)):
        cp, ci, x, _, _ = b
        h2 = torch.empty((r.forest.n_nodes, r.H), dtype=torch.float32).pin_memory()
        c2 = torch.empty_like(h2).pin_memory()
        nl = jdb.jdb_treelstm_forward_host(cp, ci, x, packed, r.D, r.H, precision, h2, c2, ws)
        assert nl == levels[k]
        assert torch.equal(b[3], h2) and torch.equal(b[4], c2), k
    # and the first and the largest request against the CPU checker
    for k in (0, int(np.argmax(sizes))):
        r = reqs[k]
        ho, co = ot.forward(r.forest.child_ptr, r.forest.child_idx, r.x_full(), r.W, r.U, r.b)
        tol = 3e-2 if r.precision == "bf16" else 1e-4
        assert np.max(np.abs(bufs[k][3].numpy() - ho)) <= tol and np.max(np.abs(bufs[k][4].numpy() - co)) <= tol


def test_an_error_stays_with_its_request_and_limits_are_enforced():
    base, reqs = _stream_of_requests(2, [6, 9, 12, 7], seed=7)
    packed = jdb.jdb_pack_weights(*(torch.from_numpy(a).to(DEV) for a in (base.W, base.U, base.b)), jdb.BF16)
    max_n = max(r.forest.n_nodes for r in reqs)
    max_e = max(r.forest.n_edges for r in reqs)
    on = jdb.Online(2, max_n, max_e, packed, base.D, base.H, jdb.BF16, jdb.BF16, DEV)
    bufs = [_request(r, pin=False) for r in reqs]      # pageable buffers work too (the copies then block)
    bad = list(bufs[1])
    ci = bad[1].clone()
    ci[0] = ci[1] if ci.numel() > 1 else 0             # a node with two parents
    bad[1] = ci
    t0 = on.submit(*bufs[0])
    t1 = on.submit(*bad)
    t2 = on.submit(*bufs[2])                           # takes slot 0 again: request 0 is completed first
    t3 = on.submit(*bufs[3])                           # takes slot 1 again: the failed request is completed first
    assert on.wait(t3) > 0 and on.wait(t2) > 0 and on.wait(t0) > 0
    with pytest.raises(jdb.JdbError) as ei:
        on.wait(t1)
    assert ei.value.status == jdb.ERR_NOT_A_FOREST
    for k in (0, 2, 3):
        r = reqs[k]
        ho, co = ot.forward(r.forest.child_ptr, r.forest.child_idx, r.x_full(), r.W, r.U, r.b)
        assert np.max(np.abs(bufs[k][3].numpy() - ho)) <= 3e-2 and np.max(np.abs(bufs[k][4].numpy() - co)) <= 3e-2
    # a request beyond the stated maximum takes no ticket; an unknown ticket is refused
    big = wl.make_workload(2, n_trees=200)
    big = wl.Workload(big.name, big.index, big.forest, big.D, big.H, big.precision, base.table, (big.token % base.table.shape[0]).astype(np.int32), base.W, base.U, base.b)
    with pytest.raises(jdb.JdbError):
        on.submit(*_request(big, pin=False))
    with pytest.raises(jdb.JdbError):
        on.wait(99)
    # an empty request completes with zero levels
    e = on.submit(torch.zeros(1, dtype=torch.int32), torch.zeros(0, dtype=torch.int32), torch.zeros((0, base.D), dtype=torch.bfloat16),
                  torch.zeros((0, base.H)), torch.zeros((0, base.H)))
    assert on.wait(e) == 0
    on.close()


@pytest.mark.parametrize("index,n_trees", [(1, 50), (2, 120), (3, 20)])
def test_roots_only_returns_the_root_rows(index, n_trees):
    """JDB_FLAG_ROOTS_ONLY: the host entries hand back the states of the roots alone, ascending by node id, bit for bit
    the rows of the full result (fp32, bf16 cooperative loop, bf16 per-level launches; ids shuffled so that roots are
    scattered over the id range)."""
    w0 = wl.make_workload(index, n_trees=n_trees, bias="random")
    forest, new_of_old = wl.relabel(w0.forest, np.random.default_rng(3))
    token = np.empty_like(w0.token)
    token[new_of_old] = w0.token
    w = wl.Workload(w0.name, w0.index, forest, w0.D, w0.H, w0.precision, w0.table, token, w0.W, w0.U, w0.b)
    f = w.forest
    precision = jdb.BF16 if w.precision == "bf16" else jdb.FP32
    packed = jdb.jdb_pack_weights(*(torch.from_numpy(a).to(DEV) for a in (w.W, w.U, w.b)), precision)
    cp, ci, x, h, c = _request(w)
    ws = jdb.forward_host_workspace(f.n_nodes, f.n_edges, w.D, w.H, precision, precision, DEV)
    jdb.jdb_treelstm_forward_host(cp, ci, x, packed, w.D, w.H, precision, h, c, ws)
    roots = np.sort(np.asarray(f.roots, dtype=np.int64))
    assert len(roots) == f.n_nodes - f.n_edges
    hr = torch.full((len(roots), w.H), float("nan")).pin_memory()
    cr = torch.full((len(roots), w.H), float("nan")).pin_memory()
    jdb.jdb_treelstm_forward_host(cp, ci, x, packed, w.D, w.H, precision, hr, cr, ws, flags=jdb.FLAG_ROOTS_ONLY)
    assert torch.equal(hr, h[roots]) and torch.equal(cr, c[roots])
    on = jdb.Online(2, f.n_nodes, f.n_edges, packed, w.D, w.H, precision, precision, DEV, flags=jdb.FLAG_ROOTS_ONLY)
    hr2, cr2 = torch.full_like(hr, float("nan")).pin_memory(), torch.full_like(cr, float("nan")).pin_memory()
    on.wait(on.submit(cp, ci, x, hr2, cr2))
    on.close()
    assert torch.equal(hr2, hr) and torch.equal(cr2, cr)
