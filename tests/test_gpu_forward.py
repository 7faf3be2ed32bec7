"""CUDA forward (through the C ABI) vs the fp64 CPU checker, element by element.

Tolerances (max-abs on h and c): 1e-4 on the fp32 path, 3e-2 on the bf16-GEMM path.  Against the
checker's bf16-matched mode (same rounding points, fp64 elsewhere) the bf16 path must be within 4e-3,
which separates rounding from mistakes: what is left there is fp32 accumulation order and the hardware
tanh approximation (about 5e-4 absolute per evaluation, a few evaluations per node, carried up the levels).
"""
import numpy as np
import pytest
import torch

from gpu_util import deliberate_trees, device_inputs, run_forward
from oracle import treelstm as ot
from paper_1904_07421_b200 import jdb
from paper_1904_07421_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-4
TOL_BF16 = 3e-2
TOL_BF16_MATCHED = 4e-3


def oracle(w, quantize=None):
    f = w.forest
    return ot.forward(f.child_ptr, f.child_idx, w.x_full(), w.W, w.U, w.b, quantize=quantize)


def matched(w, mode=jdb.MODE_AUTO):
    """The checker's bf16 mode that rounds where the kernels that will run round.  The cooperative tensor-core
    level loop (H <= 192, any mode but per-level launches) multiplies per child edge and adds the products, so only
    h_k is rounded.  The per-level launches keep a bf16 copy of every h for the recurrence and add the rounded child
    rows, rounding the sum once more.  The plain-ALU cooperative kernel (persistent mode, H > 192) rounds the sum of
    the exact rows."""
    if w.H <= 192 and mode != jdb.MODE_PER_LEVEL:
        return "bf16_edges"
    if mode == jdb.MODE_PERSISTENT:
        return "bf16"
    return "bf16_rows"


def check(w, h, c, tol, quantize=None):
    ho, co = oracle(w, quantize)
    assert np.isfinite(h).all() and np.isfinite(c).all()
    eh, ec = np.max(np.abs(h - ho)), np.max(np.abs(c - co))
    assert eh <= tol and ec <= tol, (eh, ec)
    return eh, ec


@pytest.mark.parametrize("mode", [jdb.MODE_PER_LEVEL, jdb.MODE_PERSISTENT, jdb.MODE_AUTO])
def test_config1_fp32(mode):
    w = wl.make_workload(1)
    h, c, _ = run_forward(w, mode)
    check(w, h, c, TOL_FP32)


def test_config1_fp32_nonzero_bias_relabelled_padded():
    w = wl.make_workload(1, bias="random")
    rng = np.random.default_rng(8)
    g, new_id = wl.relabel(w.forest, rng)
    tok = np.empty_like(w.token)
    tok[new_id] = w.token
    w.forest, w.token = g, tok
    h, c, _ = run_forward(w, jdb.MODE_PER_LEVEL, pad_ld=True)
    check(w, h, c, TOL_FP32)


@pytest.mark.parametrize("D,H", [(1, 1), (5, 7), (33, 31), (64, 96), (300, 150), (40, 257)])
def test_ragged_dims_and_fanouts_fp32(D, H):
    parents = [[-1], [-1, 0], [-1] + [0] * 9, [-1, 0, 1, 2, 3], [-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5],
               [-1] + [0] * 40, [-1, 0, 0, 2, 2, 2, 0]]
    w = wl.make_custom(parents, D=D, H=H, seed=100 + D + H, bias="random")
    for mode in (jdb.MODE_PER_LEVEL, jdb.MODE_PERSISTENT):
        h, c, _ = run_forward(w, mode)
        check(w, h, c, TOL_FP32)


def test_fp32_modes_agree():
    """The cooperative launch is deterministic (every K loop runs in ascending k in one thread) and the same with a
    schedule whose counts stay on the device; per-level launches sum in another order, so they agree with it to
    fp32 rounding-order noise only."""
    w = wl.make_workload(1)
    h1, c1, _ = run_forward(w, jdb.MODE_PER_LEVEL)
    h2, c2, _ = run_forward(w, jdb.MODE_PERSISTENT)
    h3, c3, _ = run_forward(w, jdb.MODE_AUTO, sync_schedule=False)
    h4, c4, _ = run_forward(w, jdb.MODE_PERSISTENT, pad_ld=True)
    assert np.array_equal(h2, h3) and np.array_equal(c2, c3)
    assert np.array_equal(h2, h4) and np.array_equal(c2, c4)
    assert np.max(np.abs(h1 - h2)) <= 1e-5 and np.max(np.abs(c1 - c2)) <= 1e-5


def test_fp32_cooperative_loop_many_children_and_plain_kernel_for_large_hidden():
    """A node with 300 children takes ten passes of the fp32 cooperative loop; H = 200 is beyond that kernel and runs
    the plain persistent kernel."""
    parents = [[-1, 0] + [1] * 300, [-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5], [-1] + list(range(40))] * 2
    for H in (70, 200):
        w = wl.make_custom(parents, D=24, H=H, seed=300 + H, bias="random")
        for pad in (False, True):
            h, c, _ = run_forward(w, jdb.MODE_PERSISTENT, pad_ld=pad)
            check(w, h, c, TOL_FP32)


@pytest.mark.parametrize("mode", [jdb.MODE_AUTO, jdb.MODE_PER_LEVEL, jdb.MODE_PERSISTENT])
@pytest.mark.parametrize("pad_ld", [False, True])
def test_config2_bf16(mode, pad_ld):
    w = wl.make_workload(2)
    h, c, _ = run_forward(w, mode, pad_ld=pad_ld)
    check(w, h, c, TOL_BF16)
    check(w, h, c, TOL_BF16_MATCHED, quantize=matched(w, mode))


def test_bf16_repeated_calls_are_deterministic():
    w = wl.make_workload(2)
    h1, c1, _ = run_forward(w, jdb.MODE_PER_LEVEL, pad_ld=True)
    h2, c2, _ = run_forward(w, jdb.MODE_PER_LEVEL, pad_ld=True)
    assert np.array_equal(h1, h2) and np.array_equal(c1, c2)


@pytest.mark.parametrize("D,H", [(8, 8), (5, 7), (64, 64), (65, 130), (300, 150), (72, 200)])
def test_ragged_dims_and_fanouts_bf16(D, H):
    parents = [[-1], [-1, 0], [-1] + [0] * 9, [-1, 0, 1, 2, 3], [-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5],
               [-1] + [0] * 140, [-1, 0, 0, 2, 2, 2, 0]] * 3
    w = wl.make_custom(parents, D=D, H=H, seed=200 + D + H, precision="bf16", bias="random")
    for pad in (False, True):
        for mode in (jdb.MODE_PER_LEVEL, jdb.MODE_PERSISTENT):   # per-level launches; one cooperative launch
            h, c, _ = run_forward(w, mode, pad_ld=pad)
            check(w, h, c, TOL_BF16_MATCHED, quantize=matched(w, mode))


def test_bf16_schedule_without_sync_feeds_every_level_loop():
    """After jdb_schedule_async the level count lives on the device only."""
    for index, trees in ((2, 64), (3, 8)):        # cooperative level loop (H <= 192); per-level launches
        w = wl.make_workload(index, n_trees=trees, bias="random")
        h, c, s = run_forward(w, jdb.MODE_AUTO, pad_ld=True, sync_schedule=False)
        assert s.n_levels == -1
        check(w, h, c, TOL_BF16_MATCHED, quantize=matched(w))


def test_bf16_plain_alu_cooperative_kernel_for_large_hidden():
    """Persistent mode with H > 192 has no tensor-core kernel and runs on the fp32 ALUs."""
    parents = [[-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5], [-1] + [0] * 12, [-1, 0, 1, 2]] * 4
    w = wl.make_custom(parents, D=40, H=200, seed=77, precision="bf16", bias="random")
    h, c, _ = run_forward(w, jdb.MODE_PERSISTENT)
    check(w, h, c, TOL_BF16_MATCHED, quantize="bf16")


def test_bf16_path_accepts_fp32_x_and_padded_rows():
    w = wl.make_workload(2, n_trees=40, bias="random")
    forest, x, packed, precision = device_inputs(w, pad_ld=True)
    sched = jdb.jdb_schedule(forest)
    h, c = jdb.jdb_treelstm_forward(forest, sched, x.float(), packed, w.D, w.H, precision)
    torch.cuda.synchronize()
    check(w, h.cpu().numpy(), c.cpu().numpy(), TOL_BF16_MATCHED, quantize=matched(w))


def test_level_ordered_outputs_through_plain_stores_agree_with_tma_stores(monkeypatch):
    """P and the bf16 copy of the leaf rows leave the GEMM epilogues as TMA stores; JDB_P_TMA=0 sends them through the
    load/store units instead.  Same arithmetic, so the results agree bit for bit, on per-level launches (H = 200: two
    hidden slices, ragged) and on the cooperative loop (H = 150).  One exception by design: in the per-level launches
    the forget sum of a node arrives as one atomic addition per group of 32 edge slots its children touch; with more
    than two groups (the 140-child roots here) the order of the additions is not fixed, so those rows are held to
    fp32 rounding-order noise instead."""
    parents = [[-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5], [-1] + [0] * 140, [-1, 0, 1, 2, 3], [-1]] * 40
    for H, mode in ((200, jdb.MODE_PER_LEVEL), (150, jdb.MODE_AUTO)):
        w = wl.make_custom(parents, D=72, H=H, seed=400 + H, precision="bf16", bias="random")
        monkeypatch.delenv("JDB_P_TMA", raising=False)
        h1, c1, _ = run_forward(w, mode, pad_ld=True)
        monkeypatch.setenv("JDB_P_TMA", "0")
        h0, c0, _ = run_forward(w, mode, pad_ld=True)
        monkeypatch.delenv("JDB_P_TMA", raising=False)
        fixed = np.diff(w.forest.child_ptr) <= 33 if mode == jdb.MODE_PER_LEVEL else np.ones(w.forest.n_nodes, dtype=bool)
        assert np.array_equal(h0[fixed], h1[fixed]) and np.array_equal(c0[fixed], c1[fixed])
        assert np.allclose(h0, h1, rtol=0, atol=2e-6) and np.allclose(c0, c1, rtol=1e-6, atol=2e-6)
        # the c of a 140-child root is a sum of 140 terms f c_k, each carrying the logistic approximation's error (up to
        # 2.6e-4 per term, measured by the test above): its bound grows with the number of children
        ho, co = oracle(w, matched(w, mode))
        fan = np.diff(w.forest.child_ptr).astype(np.float64)[:, None]
        assert np.all(np.abs(h1 - ho) <= TOL_BF16_MATCHED) and np.all(np.abs(c1 - co) <= TOL_BF16_MATCHED + 2.6e-4 * fan)


def sampled_check(index, extra_random, seed, matched_trees=None):
    """Full-size workload on the GPU in the launch configuration the benchmark times (its leading dimensions,
    automatic mode).  The checker evaluates whole trees: the ones gpu_util.deliberate_trees names (first and last tree,
    the tile that straddles the leaf/internal boundary, the last partial tile of every level, the rows on both sides
    of the 2^31 and 2^32 byte offsets) plus `extra_random` random ones; extra_random=None takes every tree.
    Everything else is held to the properties that hold at any size: finite, |h| < 1, untouched padding."""
    w = wl.make_workload(index)
    h, c, sched = run_forward(w, bench_ld=True)
    f = w.forest
    if extra_random is None:
        trees = np.arange(f.n_trees)
    else:
        trees = deliberate_trees(f, row_bytes=4 * ((w.H + 3) // 4 * 4), extra_random=extra_random, seed=seed)
        assert trees[0] == 0 and trees[-1] == f.n_trees - 1
    sub, nodes = wl.subforest(f, trees)
    x = w.x_rows(nodes)
    ho, co = ot.forward(sub.child_ptr, sub.child_idx, x, w.W, w.U, w.b)
    eh, ec = np.max(np.abs(h[nodes] - ho)), np.max(np.abs(c[nodes] - co))
    assert eh <= TOL_BF16 and ec <= TOL_BF16, (eh, ec)
    if matched_trees is not None:
        sub, nodes = wl.subforest(f, trees[:: max(1, len(trees) // matched_trees)])
        x = w.x_rows(nodes)
    hq, cq = ot.forward(sub.child_ptr, sub.child_idx, x, w.W, w.U, w.b, quantize=matched(w))
    eh, ec = np.max(np.abs(h[nodes] - hq)), np.max(np.abs(c[nodes] - cq))
    assert eh <= TOL_BF16_MATCHED and ec <= TOL_BF16_MATCHED, (eh, ec)
    assert np.isfinite(h).all() and np.isfinite(c).all()
    assert np.abs(h).max() <= 1.0
    return len(trees), len(nodes)


def test_config3_sampled():
    n_trees, _ = sampled_check(3, 600, 31)       # about 0.7 k of 4096 trees: ~10 s of checker time per mode
    assert n_trees >= 600


def test_config4_every_tree():
    sampled_check(4, None, 41, matched_trees=128)  # all 1024 trees against the plain checker (~25 s), 128 against the matched mode


def test_config5_sampled():
    n_trees, _ = sampled_check(5, 512, 51)       # at least 512 of 65536 trees: ~8 s of checker time per mode
    assert n_trees >= 512


def _variants_agree_bit_for_bit(index, tunings, n_trees=None):
    """The GEMM switches change how a product is scheduled (CTA pairs, issuer warps, launch overlap, store path, how x
    is fetched), never its arithmetic: every row of h and c must come out with the same bits.  One exception by
    design: the forget-gate GEMM adds a parent's f c_k in runs of 128 edge slots as lone CTAs and of 64 as CTA pairs, so
    the two groups of variants agree with each other to fp32 rounding order only, which a bf16 rounding of h further up
    the tree can turn into one bf16 unit in the last place of an operand: they are held to 2e-3."""
    w = wl.make_workload(index, n_trees=n_trees)
    ref = {}
    for t in tunings:
        h, c, _ = run_forward(w, bench_ld=True, tuning=t, to_host=False)
        pair_forget = t == 0 or bool(t & jdb.TUNE_PAIR_FORGET)
        if pair_forget not in ref:
            ref[pair_forget] = (h, c, t)
            continue
        assert torch.equal(h, ref[pair_forget][0]) and torch.equal(c, ref[pair_forget][1]), (t, ref[pair_forget][2])
        del h, c
    if len(ref) == 2:
        assert float((ref[True][0] - ref[False][0]).abs().max()) <= 2e-3 and float((ref[True][1] - ref[False][1]).abs().max()) <= 2e-3
    h, c, _ = ref[True] if True in ref else ref[False]
    return w, h, c


_TUNINGS = [jdb.TUNE_SET,                                                          # lone CTAs everywhere
            0,                                                                     # the defaults
            jdb.TUNE_SET | jdb.TUNE_PAIR_XPROJ | jdb.TUNE_PAIR_LEVEL | jdb.TUNE_PAIR_FORGET,   # CTA pairs wherever allowed
            jdb.TUNE_SET | jdb.TUNE_PAIR_FORGET | jdb.TUNE_TWO_ISSUERS,
            jdb.TUNE_SET | jdb.TUNE_PAIR_FORGET | jdb.TUNE_NO_PDL,
            jdb.TUNE_SET | jdb.TUNE_PAIR_XPROJ | jdb.TUNE_PLAIN_STORES,
            jdb.TUNE_SET | jdb.TUNE_PAIR_FORGET | jdb.TUNE_GATHER_X,
            jdb.TUNE_SET | jdb.TUNE_PAIR_XPROJ | jdb.TUNE_GATHER_X | jdb.TUNE_TWO_ISSUERS]



def test_config3_gemm_variants_agree_on_every_row():
    _variants_agree_bit_for_bit(3, _TUNINGS)


def test_config5_gemm_variants_agree_on_every_row():
    """1.57 M rows each; the CTA-pair kernels are reached only by forests of this size."""
    w, h, c = _variants_agree_bit_for_bit(5, _TUNINGS)
    # and one of them (all agree) against the checker on a few trees
    trees = deliberate_trees(w.forest, row_bytes=4 * w.H, extra_random=32, seed=52)
    sub, nodes = wl.subforest(w.forest, trees)
    ho, co = ot.forward(sub.child_ptr, sub.child_idx, w.x_rows(nodes), w.W, w.U, w.b)
    idx = torch.from_numpy(nodes).to(h.device)
    assert np.max(np.abs(h[idx].cpu().numpy() - ho)) <= TOL_BF16 and np.max(np.abs(c[idx].cpu().numpy() - co)) <= TOL_BF16


def test_fast_tanh_and_sigmoid_error_measured_through_the_library():
    """The bf16 path evaluates tanh with the hardware approximation and the logistic function as
    0.5 + 0.5 tanh(t / 2).  Leaves make both observable from outside: with z_i = 0 the cell state of a leaf is
    c = 0.5 tanh(z_u) exactly (0.5 is what the logistic form gives at 0), and with z_u constant it is
    c = sigma(z_i) * T with T = tanh(z_u) read off the first kind of leaf.  Pre-activations are swept over
    [-10, 10] on values that bfloat16 holds exactly (x = t, weight 1: the product is exact).  The bounds are the
    ones the tolerances are derived from: 5e-4 absolute for tanh, half of that for the logistic function."""
    steps = np.arange(-10.0, 10.0 + 1e-9, 1.0 / 64.0)
    t = wl.round_to_bf16(steps.astype(np.float32)).astype(np.float64)
    t = np.unique(np.concatenate([t, [2.0]]))
    n = len(t)
    D, H = 2, 2
    forest = jdb.forest_to_device(np.zeros(n + 1, dtype=np.int32), np.zeros(0, dtype=np.int32))
    x = torch.zeros((n, 8), dtype=torch.bfloat16, device="cuda")
    x[:, 0] = torch.from_numpy(t).to(torch.bfloat16)
    x[:, 1] = 1.0
    W = np.zeros((4 * H, D), dtype=np.float32)
    b = np.zeros(4 * H, dtype=np.float32)
    W[2 * H + 0, 0] = 1.0          # hidden unit 0: z_i = 0, z_u = t
    W[0 * H + 1, 0] = 1.0          # hidden unit 1: z_i = t, z_u = 2 (through the constant input column)
    W[2 * H + 1, 1] = 2.0
    U = np.zeros((4 * H, H), dtype=np.float32)
    packed = jdb.jdb_pack_weights(*(torch.from_numpy(a).cuda() for a in (W, U, b)), jdb.BF16)
    sched = jdb.jdb_schedule(forest)
    h, c = jdb.jdb_treelstm_forward(forest, sched, x, packed, D, H, jdb.BF16)
    torch.cuda.synchronize()
    c = c.cpu().numpy().astype(np.float64)
    tanh_fast = 2.0 * c[:, 0]
    err_tanh = np.max(np.abs(tanh_fast - np.tanh(t)))
    T = tanh_fast[np.nonzero(t == 2.0)[0][0]]
    sig_fast = c[:, 1] / T
    err_sig = np.max(np.abs(sig_fast - 1.0 / (1.0 + np.exp(-t))))
    assert err_tanh <= 5e-4, err_tanh
    assert err_sig <= 2.6e-4, err_sig
    assert err_tanh > 0          # it IS an approximation; an exact result would mean the test looks at the wrong thing


def test_very_wide_level_in_the_cooperative_loop():
    """A forest whose first level above the leaves is very wide (70000 two-leaf parents) over a few deeper trees: the
    analysis reports the wide level, and the cooperative loop (H <= 192) evaluates it like any other, from a
    schedule whose counts are on the host and from one whose counts stay on the device, with the same bits."""
    deep = [-1, 0, 0, 1, 1, 2, 3, 3, 5, 6, 6, 8]
    parents = [[-1, 0, 0]] * 70000 + [deep] * 300
    w = wl.make_custom(parents, D=16, H=40, seed=9, precision="bf16", bias="random")
    h1, c1, s1 = run_forward(w, pad_ld=True)
    assert s1.n_wide_levels == 1 and s1.n_levels > 3
    h2, c2, s2 = run_forward(w, pad_ld=True, sync_schedule=False)
    assert s2.n_wide_levels == -1
    assert np.array_equal(h1, h2) and np.array_equal(c1, c2)
    trees = np.concatenate([np.arange(0, 70000, 1000), np.arange(70000, 70300, 10)])
    sub, nodes = wl.subforest(w.forest, trees)
    x = w.x_rows(nodes)
    ho, co = ot.forward(sub.child_ptr, sub.child_idx, x, w.W, w.U, w.b)
    assert np.max(np.abs(h1[nodes] - ho)) <= TOL_BF16 and np.max(np.abs(c1[nodes] - co)) <= TOL_BF16
    hq, cq = ot.forward(sub.child_ptr, sub.child_idx, x, w.W, w.U, w.b, quantize="bf16_edges")
    assert np.max(np.abs(h1[nodes] - hq)) <= TOL_BF16_MATCHED and np.max(np.abs(c1[nodes] - cq)) <= TOL_BF16_MATCHED
    # the same forest through the per-level launches: 140000 edge slots on level 1
    h3, c3, _ = run_forward(w, jdb.MODE_PER_LEVEL, pad_ld=True)
    hq, cq = ot.forward(sub.child_ptr, sub.child_idx, x, w.W, w.U, w.b, quantize="bf16_rows")
    assert np.max(np.abs(h3[nodes] - hq)) <= TOL_BF16_MATCHED and np.max(np.abs(c3[nodes] - cq)) <= TOL_BF16_MATCHED
    assert np.max(np.abs(h3 - h1)) <= 2e-2


def test_empty_forest_and_argument_errors():
    import ctypes as C
    w = wl.make_workload(1, n_trees=3)
    forest, x, packed, precision = device_inputs(w)
    sched = jdb.jdb_schedule(forest)
    L = jdb.lib()
    cf, cs = forest.c(), sched.c()
    opts = jdb.COpts(precision, 0, 0, 0, 0, None, None, None, None, 0)
    h = torch.empty((forest.n_nodes, w.H), device="cuda")
    ws = jdb.forward_workspace(forest, sched, w.D, w.H, precision)
    vp = lambda t: C.c_void_p(t.data_ptr())
    call = lambda **kw: L.jdb_treelstm_forward(
        C.byref(cf), C.byref(cs), vp(x), kw.get("xd", jdb.FP32), kw.get("ldx", w.D), vp(packed), w.D, w.H, vp(h), vp(h),
        kw.get("ldh", w.H), C.byref(kw.get("opts", opts)), vp(ws), kw.get("wsb", ws.numel()), None)
    assert call(ldx=w.D - 1) == jdb.ERR_INVALID_ARG
    assert call(ldh=w.H - 1) == jdb.ERR_INVALID_ARG
    assert call(xd=jdb.BF16) == jdb.ERR_INVALID_ARG      # fp32 precision needs fp32 x
    assert call(wsb=16) == jdb.ERR_WORKSPACE
    assert call(opts=jdb.COpts(7, 0, 0, 0, 0, None, None, None, None, 0)) == jdb.ERR_INVALID_ARG
    empty = jdb.forest_to_device([0], [])
    se = jdb.jdb_schedule(empty)
    assert se.n_levels == 0
    he, ce = jdb.jdb_treelstm_forward(empty, se, x, packed, w.D, w.H, precision)
    assert he.shape[0] == 0


@pytest.mark.parametrize("index,trees,H_override", [(2, 64, None), (3, 24, None), (1, 16, None), (2, 40, 200)])
def test_host_buffer_entry_point(index, trees, H_override):
    """Host buffers in, host buffers out: the cooperative bf16 loop (workload 2), per-level launches with H > 192
    (workload 3, and H = 200 with ragged slices), and the fp32 path (workload 1)."""
    if H_override is None:
        w = wl.make_workload(index, n_trees=trees, bias="random")
    else:
        base = wl.make_workload(index, n_trees=trees)
        w = wl.make_custom([wl.parent_array(wl.subforest(base.forest, [t])[0]) for t in range(trees)], D=72, H=H_override,
                           seed=17, precision="bf16", bias="random")
    f = w.forest
    precision = jdb.BF16 if w.precision == "bf16" else jdb.FP32
    dt = torch.bfloat16 if precision == jdb.BF16 else torch.float32
    packed = device_inputs(w)[2]
    x = torch.from_numpy(w.x_full()).to(dt).pin_memory()
    cp = torch.from_numpy(f.child_ptr).pin_memory()
    ci = torch.from_numpy(f.child_idx).pin_memory()
    h = torch.empty((f.n_nodes, w.H), dtype=torch.float32).pin_memory()
    c = torch.empty((f.n_nodes, w.H), dtype=torch.float32).pin_memory()
    ws = jdb.forward_host_workspace(f.n_nodes, f.n_edges, w.D, w.H, precision, precision)
    n_levels = jdb.jdb_treelstm_forward_host(cp, ci, x, packed, w.D, w.H, precision, h, c, ws)
    from oracle import schedule as osched
    assert n_levels == osched.schedule(f.child_ptr, f.child_idx, f.n_nodes)[4]
    if precision == jdb.FP32:
        check(w, h.numpy(), c.numpy(), TOL_FP32)
    else:
        check(w, h.numpy(), c.numpy(), TOL_BF16)
        check(w, h.numpy(), c.numpy(), TOL_BF16_MATCHED, quantize=matched(w))


def test_step_plan_with_deferred_status_matches_the_plain_calls():
    w = wl.make_workload(2, n_trees=96, bias="random")
    forest, x, packed, precision = device_inputs(w, pad_ld=True)
    sched = jdb.alloc_schedule(forest.n_nodes)
    sws = jdb.schedule_workspace(forest)
    fws = jdb.forward_workspace(forest, sched, w.D, w.H, precision)      # sized without knowing the leaf count
    h = torch.empty((forest.n_nodes, 152), device="cuda")
    c = torch.empty_like(h)
    plan = jdb.StepPlan(forest, sched, sws, x, packed, w.D, w.H, precision, h, c, fws)
    for _ in range(3):
        plan.run()
    n_levels, n_leaves = plan.status()
    ref = jdb.jdb_schedule(forest)
    assert (n_levels, n_leaves) == (ref.n_levels, ref.n_leaves)
    check(w, h[:, :w.H].cpu().numpy(), c[:, :w.H].cpu().numpy(), TOL_BF16_MATCHED, quantize=matched(w))


def test_deferred_status_reports_a_malformed_forest():
    w = wl.make_workload(2, n_trees=32)
    cp, ci = w.forest.child_ptr.copy(), w.forest.child_idx.copy()
    ci[3] = ci[4]                                                         # a node with two parents
    forest = jdb.forest_to_device(cp, ci)
    _, x, packed, precision = device_inputs(w, pad_ld=True)
    sched = jdb.alloc_schedule(forest.n_nodes)
    h = torch.zeros((forest.n_nodes, 152), device="cuda")
    c = torch.zeros_like(h)
    plan = jdb.StepPlan(forest, sched, jdb.schedule_workspace(forest), x, packed, w.D, w.H, precision, h, c,
                        jdb.forward_workspace(forest, sched, w.D, w.H, precision))
    plan.run()                                                             # enqueues; nothing is reported yet
    with pytest.raises(jdb.JdbError) as ei:
        plan.status()
    assert ei.value.status == jdb.ERR_NOT_A_FOREST


def test_level_barrier_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    """A grid barrier whose wait limit is 1 ns: the CTAs of a light tile give up waiting for the CTAs of a heavy
    one (a node with 6000 children), every CTA leaves the kernel, and the call returns JDB_ERR_TIMEOUT.
    Nothing hangs: the wait is bounded by construction, this only makes the bound tiny."""
    star = [-1, 0] + [1] * 6000                    # root -> hub -> 6000 leaves: depths 2, 1, 0
    chains = [[-1, 0, 1]] * 40                     # forty short chains: more nodes at levels 1 and 2
    w = wl.make_custom([star] + chains, D=16, H=64, seed=5, precision="bf16", bias="random")
    forest, x, packed, precision = device_inputs(w, pad_ld=True)
    sched = jdb.jdb_schedule(forest)
    assert sched.n_levels == 3
    with pytest.raises(jdb.JdbError) as ei:
        jdb.jdb_treelstm_forward(forest, sched, x, packed, w.D, w.H, precision, mode=jdb.MODE_PERSISTENT,
                                 barrier_timeout_ns=1)
    assert ei.value.status == jdb.ERR_TIMEOUT
    torch.cuda.synchronize()
    # same call with the default limit: correct results on the same context (the hub's c is a sum of 6000 terms,
    # so its error is taken relative to its size)
    h, c = jdb.jdb_treelstm_forward(forest, sched, x, packed, w.D, w.H, precision, mode=jdb.MODE_PERSISTENT)
    torch.cuda.synchronize()
    ho, co = oracle(w, matched(w, jdb.MODE_PERSISTENT))
    assert np.all(np.abs(h.cpu().numpy() - ho) <= TOL_BF16_MATCHED + 1e-2 * np.abs(ho))
    assert np.all(np.abs(c.cpu().numpy() - co) <= TOL_BF16_MATCHED + 1e-2 * np.abs(co))


@pytest.mark.parametrize("mode", [jdb.MODE_PER_LEVEL, jdb.MODE_PERSISTENT])
def test_bf16_degenerate_forests(mode):
    """One node; leaves only (a single level); one long chain (one node per level)."""
    for parents in ([[-1]], [[-1]] * 300, [[-1] + list(range(130))]):
        w = wl.make_custom(parents, D=24, H=40, seed=len(parents) + len(parents[0]), precision="bf16", bias="random")
        h, c, s = run_forward(w, mode, pad_ld=True)
        assert s.n_levels == (1 if len(parents[0]) == 1 else 131)
        check(w, h, c, TOL_BF16_MATCHED, quantize=matched(w, mode))


_DEBUG_CASES = [("fp32", jdb.MODE_PER_LEVEL, 70), ("fp32", jdb.MODE_PERSISTENT, 70), ("fp32", jdb.MODE_PERSISTENT, 200),
                ("bf16", jdb.MODE_AUTO, 150), ("bf16", jdb.MODE_PER_LEVEL, 150), ("bf16", jdb.MODE_AUTO, 200),
                ("bf16", jdb.MODE_PERSISTENT, 200)]


@pytest.mark.parametrize("precision,mode,H", _DEBUG_CASES)
def test_debug_checks_pass_on_every_path_and_change_nothing(precision, mode, H):
    """JDB_FLAG_DEBUG_CHECKS makes every kernel hold the indices it follows against the sizes of the arrays they
    index.  On a consistent forest and schedule nothing is reported, on every level-loop variant, and the results are
    the ones of the unchecked run."""
    parents = [[-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5], [-1] + [0] * 40, [-1, 0, 1, 2, 3], [-1], [-1] + list(range(20))] * 30
    w = wl.make_custom(parents, D=40, H=H, seed=600 + H, precision=precision, bias="random")
    rng = np.random.default_rng(3)
    g, new_id = wl.relabel(w.forest, rng)
    tok = np.empty_like(w.token)
    tok[new_id] = w.token
    w.forest, w.token = g, tok
    h0, c0, _ = run_forward(w, mode, pad_ld=True)
    h1, c1, s = run_forward(w, mode, pad_ld=True, flags=jdb.FLAG_DEBUG_CHECKS)
    assert jdb.jdb_debug_report(s)[0] == 0
    assert np.allclose(h0, h1, rtol=0, atol=2e-6) and np.allclose(c0, c1, rtol=1e-6, atol=2e-6)
    check(w, h1, c1, TOL_FP32 if precision == "fp32" else TOL_BF16)


@pytest.mark.parametrize("precision,mode,H", _DEBUG_CASES)
def test_debug_checks_report_a_schedule_that_does_not_fit_the_forest(precision, mode, H):
    """A schedule made for a forest of N nodes, handed in with a forest header that claims N - 7: the schedule's level
    offsets and node ids then point past what the header allows.  With the checks on, the call reports
    JDB_ERR_CHECK and names the offender instead of following it.  (Every buffer here is allocated for the full N, so
    nothing could leave its allocation even unchecked.)"""
    parents = [[-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5], [-1] + [0] * 40, [-1, 0, 1, 2, 3]] * 30
    w = wl.make_custom(parents, D=40, H=H, seed=700 + H, precision=precision, bias="random")
    forest, x, packed, prec = device_inputs(w, pad_ld=True)
    sched = jdb.jdb_schedule(forest)
    n = forest.n_nodes
    ws = torch.empty(2 * jdb.forward_workspace(forest, sched, w.D, w.H, prec).numel() + (1 << 20), dtype=torch.uint8, device="cuda")
    h = torch.zeros((n, w.H + 2), device="cuda")
    c = torch.zeros_like(h)
    short = jdb.Forest(forest.child_ptr, forest.child_idx, n - 7, forest.n_edges)
    with pytest.raises(jdb.JdbError) as ei:
        jdb.jdb_treelstm_forward(short, sched, x, packed, w.D, w.H, prec, mode=mode, h=h, c=c, ws=ws,
                                 flags=jdb.FLAG_DEBUG_CHECKS)
    assert ei.value.status == jdb.ERR_CHECK
    what, value, bound, where = jdb.jdb_debug_report(sched)
    assert what != 0 and not (0 <= value < bound)
    torch.cuda.synchronize()
    # the same buffers with the true header: clean
    hh, cc = jdb.jdb_treelstm_forward(forest, sched, x, packed, w.D, w.H, prec, mode=mode, h=h, c=c, ws=ws,
                                      flags=jdb.FLAG_DEBUG_CHECKS)
    torch.cuda.synchronize()
    assert jdb.jdb_debug_report(sched)[0] == 0
    check(w, hh[:, :w.H].cpu().numpy(), cc[:, :w.H].cpu().numpy(), TOL_FP32 if precision == "fp32" else TOL_BF16)


def test_tree_partitioned_cooperative_loop_agrees_bit_for_bit_with_grid_barriers():
    """The cooperative bf16 loop ends every level in a barrier over the whole grid, or (JDB_TUNE_TREE_GROUPS) partitions
    the forest by tree over its groups of CTAs, which then synchronise inside a group only.  A node's arithmetic does
    not depend on which tile it shares with whom, so both give the same bits: on a deep forest and on small ragged
    ones."""
    w = wl.make_workload(4, n_trees=256)
    h0, c0, _ = run_forward(w, pad_ld=True)
    h1, c1, _ = run_forward(w, pad_ld=True, tuning=jdb.TUNE_SET | jdb.TUNE_TREE_GROUPS)
    h2, c2, _ = run_forward(w, pad_ld=True, tuning=jdb.TUNE_SET | jdb.TUNE_TREE_GROUPS, flags=jdb.FLAG_DEBUG_CHECKS)
    assert np.array_equal(h0, h1) and np.array_equal(c0, c1) and np.array_equal(h0, h2) and np.array_equal(c0, c2)
    check(w, h1, c1, TOL_BF16_MATCHED, quantize=matched(w))
    parents = [[-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5], [-1] + [0] * 140, [-1, 0, 1, 2, 3], [-1], [-1] + list(range(60))] * 40
    for H in (40, 150):
        w = wl.make_custom(parents, D=72, H=H, seed=800 + H, precision="bf16", bias="random")
        rng = np.random.default_rng(H)
        g, new_id = wl.relabel(w.forest, rng)
        tok = np.empty_like(w.token)
        tok[new_id] = w.token
        w.forest, w.token = g, tok
        h0, c0, _ = run_forward(w, pad_ld=True)
        h1, c1, _ = run_forward(w, pad_ld=True, tuning=jdb.TUNE_SET | jdb.TUNE_TREE_GROUPS)
        assert np.array_equal(h0, h1) and np.array_equal(c0, c1)
        check(w, h1, c1, TOL_BF16_MATCHED, quantize=matched(w))


@pytest.mark.parametrize("D,H", [(40, 200), (97, 257), (64, 512)])
def test_fp32_large_hidden_size_runs_through_the_gemm_levels(D, H):
    """fp32 with H > 192 and a synchronised schedule goes level by level through the tiled GEMM; the same call with
    JDB_FLAG_NO_SYNC keeps the plain-ALU cooperative kernel.  Both against the checker (1e-4) and against each other."""
    parents = [[-1, 0, 0, 1, 1, 1, 2, 5, 5, 5, 5], [-1] + [0] * 140, [-1, 0, 1, 2, 3], [-1], [-1] + list(range(20))] * 12
    w = wl.make_custom(parents, D=D, H=H, seed=900 + H, precision="fp32", bias="random")
    g, new_id = wl.relabel(w.forest, np.random.default_rng(4))
    tok = np.empty_like(w.token)
    tok[new_id] = w.token
    w.forest, w.token = g, tok
    h0, c0, _ = run_forward(w, pad_ld=True)
    check(w, h0, c0, TOL_FP32)
    h1, c1, s = run_forward(w, pad_ld=True, flags=jdb.FLAG_NO_SYNC)
    assert jdb.jdb_sched_status(s)[0] > 0
    assert np.max(np.abs(h0 - h1)) <= 2e-5 and np.max(np.abs(c0 - c1)) <= 2e-5
