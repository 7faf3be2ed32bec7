"""Relatedness head on the GPU (through the C ABI) against the fp64 checker, on root states the library computed."""
import numpy as np
import pytest
import torch

from gpu_util import run_forward
from oracle import relatedness as orl
from paper_1904_07421_b200 import jdb
from paper_1904_07421_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("index,trees,Hs,K", [(2, 256, 50, 5), (1, 64, 37, 5), (3, 64, 64, 7)])
def test_head_matches_the_checker(index, trees, Hs, K):
    w = wl.make_workload(index, n_trees=trees)
    h, _, _ = run_forward(w, to_host=False)
    H = w.H
    rng = np.random.default_rng(40 + index)
    Wx, Wp = rng.uniform(-0.3, 0.3, (Hs, H)).astype(np.float32), rng.uniform(-0.3, 0.3, (Hs, H)).astype(np.float32)
    bh, Wq, bq = (rng.uniform(-0.5, 0.5, s).astype(np.float32) for s in ((Hs,), (K, Hs), (K,)))
    roots = w.forest.roots.astype(np.int64)
    left, right = roots[0::2], roots[1::2]                     # consecutive trees form a pair, as sentence pairs do
    left, right = np.concatenate([left, roots[:3]]), np.concatenate([right, roots[:3]])   # and three trees against themselves
    dev = lambda a: torch.from_numpy(a).cuda()
    y, p, bad = jdb.jdb_relatedness_head(h, dev(left), dev(right), dev(Wx), dev(Wp), dev(bh), dev(Wq), dev(bq))
    torch.cuda.synchronize()
    assert int(bad.item()) == 0
    yo, po = orl.head(h.cpu().numpy(), left, right, Wx, Wp, bh, Wq, bq)     # same root states: only the head is compared
    assert np.max(np.abs(y.cpu().numpy() - yo)) <= 2e-5 and np.max(np.abs(p.cpu().numpy() - po)) <= 1e-5
    assert np.allclose(p.sum(dim=1).cpu().numpy(), 1.0, atol=1e-5)


def test_head_edge_cases():
    h = torch.randn(10, 12, device="cuda")
    W = torch.randn(4, 12, device="cuda")
    b, Wq, bq = torch.randn(4, device="cuda"), torch.randn(5, 4, device="cuda"), torch.randn(5, device="cuda")
    idx = lambda *v: torch.tensor(v, dtype=torch.int32, device="cuda")
    y, p, bad = jdb.jdb_relatedness_head(h, idx(), idx(), W, W, b, Wq, bq)                   # no pairs
    assert y.numel() == 0
    y, p, bad = jdb.jdb_relatedness_head(h, idx(0, 11, 3), idx(1, 2, -1), W, W, b, Wq, bq)  # two root ids out of range
    torch.cuda.synchronize()
    assert int(bad.item()) == 1
    yo, _ = orl.head(h.cpu().numpy(), [0], [1], W.cpu().numpy(), W.cpu().numpy(), b.cpu().numpy(), Wq.cpu().numpy(), bq.cpu().numpy())
    assert abs(float(y[0]) - yo[0]) <= 2e-5
    with pytest.raises(jdb.JdbError) as ei:
        jdb.jdb_relatedness_head(h, idx(0), idx(1), W, W, b, torch.randn(40, 4, device="cuda"), torch.randn(40, device="cuda"))
    assert ei.value.status == jdb.ERR_UNSUPPORTED
