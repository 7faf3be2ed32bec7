"""Thin ctypes binding over libjdb (include/jdb.h).  Argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory; every step of the
path runs inside the library's kernels.  There is no CPU fallback: if the library
has not been built, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libjdb.so")

OK, ERR_INVALID_ARG, ERR_NOT_A_FOREST, ERR_WORKSPACE, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_CHECK = range(8)
FP32, BF16 = 0, 1
FLAG_NO_SYNC, FLAG_DEBUG_CHECKS, FLAG_ROOTS_ONLY = 1, 2, 4
TUNE_SET, TUNE_PAIR_XPROJ, TUNE_PAIR_LEVEL, TUNE_PAIR_FORGET, TUNE_TWO_ISSUERS, TUNE_NO_PDL, TUNE_PLAIN_STORES = 1, 2, 4, 8, 16, 32, 64
TUNE_GATHER_X, TUNE_TREE_GROUPS = 128, 256
MODE_AUTO, MODE_PER_LEVEL, MODE_PERSISTENT = 0, 1, 2
META_INTS = 16

EXPORTS = [
    "jdb_status_string", "jdb_last_cuda_error", "jdb_schedule_workspace_bytes", "jdb_schedule",
    "jdb_schedule_async", "jdb_schedule_static", "jdb_packed_weights_bytes", "jdb_pack_weights", "jdb_forward_workspace_bytes",
    "jdb_treelstm_forward", "jdb_sched_status", "jdb_debug_report", "jdb_forward_host_workspace_bytes",
    "jdb_treelstm_forward_host", "jdb_launch_counts_workspace_bytes", "jdb_launch_counts", "jdb_relatedness_head",
    "jdb_treelstm_backward_workspace_bytes", "jdb_treelstm_backward",
    "jdb_batch_plan_workspace_bytes", "jdb_batch_plan", "jdb_cells_forward_workspace_bytes", "jdb_cells_forward",
    "jdb_online_workspace_bytes", "jdb_online_create", "jdb_online_submit", "jdb_online_wait", "jdb_online_destroy",
]
CELL_CHILDSUM, CELL_NARY = 0, 1


class CForest(C.Structure):
    _fields_ = [("child_ptr", C.c_void_p), ("child_idx", C.c_void_p), ("n_nodes", C.c_int32), ("n_edges", C.c_int32)]


class CSched(C.Structure):
    _fields_ = [("depth", C.c_void_p), ("level_ptr", C.c_void_p), ("perm", C.c_void_p), ("meta", C.c_void_p),
                ("n_levels", C.c_int32), ("n_leaves", C.c_int32), ("n_wide_levels", C.c_int32), ("reserved0", C.c_int32)]


class COpts(C.Structure):
    _fields_ = [("precision", C.c_int32), ("mode", C.c_int32), ("flags", C.c_int32), ("tuning", C.c_int32),
                ("barrier_timeout_ns", C.c_uint64), ("ev_begin", C.c_void_p), ("ev_xproj_done", C.c_void_p),
                ("ev_levels_done", C.c_void_p), ("trace", C.c_void_p), ("trace_cap", C.c_int64)]


class CLaunchStats(C.Structure):
    _fields_ = [("cells_unbatched", C.c_int64), ("cells_batched", C.c_int64), ("ops_unbatched", C.c_int64),
                ("ops_batched", C.c_int64), ("n_levels", C.c_int32), ("reserved", C.c_int32)]


class JdbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().jdb_status_string(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError {lib().jdb_last_cuda_error()})"
        super().__init__(f"{where}: {msg}")


_lib = None


def lib():
    """The loaded C library; raises if it was never built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1904_07421_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    L.jdb_status_string.restype = C.c_char_p
    L.jdb_status_string.argtypes = [C.c_int]
    L.jdb_last_cuda_error.restype = C.c_int
    L.jdb_schedule_workspace_bytes.restype = sz
    L.jdb_schedule_workspace_bytes.argtypes = [i32, i32]
    for name in ("jdb_schedule", "jdb_schedule_async"):
        fn = getattr(L, name)
        fn.restype = C.c_int
        fn.argtypes = [C.POINTER(CForest), C.POINTER(CSched), vp, sz, vp]
    L.jdb_schedule_static.restype = C.c_int
    L.jdb_schedule_static.argtypes = [C.POINTER(CForest), C.POINTER(CSched), vp]
    L.jdb_packed_weights_bytes.restype = sz
    L.jdb_packed_weights_bytes.argtypes = [i32, i32, i32]
    L.jdb_pack_weights.restype = C.c_int
    L.jdb_pack_weights.argtypes = [vp, vp, vp, i32, i32, i32, vp, sz, vp]
    L.jdb_forward_workspace_bytes.restype = sz
    L.jdb_forward_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    L.jdb_treelstm_forward.restype = C.c_int
    L.jdb_treelstm_forward.argtypes = [C.POINTER(CForest), C.POINTER(CSched), vp, i32, i64, vp, i32, i32, vp, vp, i64,
                                       C.POINTER(COpts), vp, sz, vp]
    L.jdb_sched_status.restype = C.c_int
    L.jdb_sched_status.argtypes = [C.POINTER(CSched), C.POINTER(i32), C.POINTER(i32), vp]
    L.jdb_debug_report.restype = C.c_int
    L.jdb_debug_report.argtypes = [C.POINTER(CSched), C.POINTER(i32 * 4), vp]
    L.jdb_launch_counts_workspace_bytes.restype = sz
    L.jdb_launch_counts_workspace_bytes.argtypes = [i32]
    L.jdb_launch_counts.restype = C.c_int
    L.jdb_launch_counts.argtypes = [C.POINTER(CForest), C.POINTER(CSched), C.POINTER(CLaunchStats), vp, sz, vp]
    L.jdb_treelstm_backward_workspace_bytes.restype = C.c_size_t
    L.jdb_treelstm_backward_workspace_bytes.argtypes = [i32, i32, i32, i32]
    L.jdb_treelstm_backward.restype = C.c_int
    L.jdb_treelstm_backward.argtypes = [vp, vp, vp, i64, vp, vp, vp, i32, i32, vp, vp, i64, vp, vp, i64, vp, vp, vp, vp, i64,
                                        vp, C.c_size_t, vp]
    L.jdb_batch_plan_workspace_bytes.restype = C.c_size_t
    L.jdb_batch_plan_workspace_bytes.argtypes = [i32]
    L.jdb_batch_plan.restype = C.c_int
    L.jdb_batch_plan.argtypes = [vp, vp, vp, i32, vp, vp, C.c_size_t, vp]
    L.jdb_cells_forward_workspace_bytes.restype = C.c_size_t
    L.jdb_cells_forward_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    L.jdb_cells_forward.restype = C.c_int
    L.jdb_cells_forward.argtypes = [vp, vp, vp, vp, i32, vp, i64, i32, i32, vp, vp, i64, vp, C.c_size_t, vp]
    L.jdb_online_workspace_bytes.restype = C.c_size_t
    L.jdb_online_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32, i32]
    L.jdb_online_create.restype = C.c_int
    L.jdb_online_create.argtypes = [vp, i32, i32, i32, vp, i32, i32, vp, i32, vp, C.c_size_t]
    L.jdb_online_submit.restype = C.c_int
    L.jdb_online_submit.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp]
    L.jdb_online_wait.restype = C.c_int
    L.jdb_online_wait.argtypes = [vp, i64, vp]
    L.jdb_online_destroy.restype = C.c_int
    L.jdb_online_destroy.argtypes = [vp]
    L.jdb_relatedness_head.restype = C.c_int
    L.jdb_relatedness_head.argtypes = [vp, i64, i32, vp, vp, i32, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp]
    L.jdb_forward_host_workspace_bytes.restype = sz
    L.jdb_forward_host_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32]
    L.jdb_treelstm_forward_host.restype = C.c_int
    L.jdb_treelstm_forward_host.argtypes = [vp, vp, i32, i32, vp, i32, vp, i32, i32, vp, vp, C.POINTER(COpts), vp, sz,
                                            C.POINTER(i32), vp]
    _lib = L
    return L


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _device_bytes(n: int, device) -> torch.Tensor:
    # torch's caching allocator returns 512-byte aligned blocks
    return torch.empty(max(int(n), 256), dtype=torch.uint8, device=device)


@dataclass
class Forest:
    child_ptr: torch.Tensor  # int32 [n_nodes + 1] cuda
    child_idx: torch.Tensor  # int32 [n_edges] cuda
    n_nodes: int
    n_edges: int

    def c(self) -> CForest:
        return CForest(self.child_ptr.data_ptr() if self.child_ptr.numel() else None,
                       self.child_idx.data_ptr() if self.child_idx.numel() else None, self.n_nodes, self.n_edges)


def forest_to_device(child_ptr, child_idx, device="cuda") -> Forest:
    cp = torch.as_tensor(child_ptr, dtype=torch.int32).to(device).contiguous()
    ci = torch.as_tensor(child_idx, dtype=torch.int32).to(device).contiguous()
    return Forest(cp, ci, int(cp.numel() - 1), int(ci.numel()))


@dataclass
class Schedule:
    depth: torch.Tensor
    level_ptr: torch.Tensor   # capacity n_nodes + 2; entries 0..n_levels valid
    perm: torch.Tensor
    meta: torch.Tensor
    n_levels: int
    n_leaves: int
    n_wide_levels: int = -1   # leading levels (from level 1) of at least 65536 nodes; -1 when unknown on the host

    def c(self) -> CSched:
        return CSched(self.depth.data_ptr(), self.level_ptr.data_ptr(), self.perm.data_ptr(), self.meta.data_ptr(),
                      self.n_levels, self.n_leaves, self.n_wide_levels, 0)


def alloc_schedule(n_nodes: int, device="cuda") -> Schedule:
    n = max(n_nodes, 1)
    return Schedule(torch.empty(n, dtype=torch.int32, device=device),
                    torch.empty(n + 2, dtype=torch.int32, device=device),
                    torch.empty(n, dtype=torch.int32, device=device),
                    torch.zeros(META_INTS, dtype=torch.int32, device=device), -1, -1)


def schedule_workspace(forest: Forest) -> torch.Tensor:
    return _device_bytes(lib().jdb_schedule_workspace_bytes(forest.n_nodes, forest.n_edges), forest.child_ptr.device)


def jdb_schedule(forest: Forest, out: Optional[Schedule] = None, ws: Optional[torch.Tensor] = None,
                 stream=None, sync: bool = True) -> Schedule:
    """depth, level_ptr, perm of the forest (Section 4.2's depth table)."""
    out = alloc_schedule(forest.n_nodes, forest.child_ptr.device) if out is None else out
    ws = schedule_workspace(forest) if ws is None else ws
    cf, cs = forest.c(), out.c()
    fn = lib().jdb_schedule if sync else lib().jdb_schedule_async
    st = fn(C.byref(cf), C.byref(cs), _ptr(ws), ws.numel(), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_schedule")
    out.n_levels, out.n_leaves, out.n_wide_levels = cs.n_levels, cs.n_leaves, cs.n_wide_levels
    return out


STATIC_MAX_NODES = 65536


def jdb_schedule_static(forest: Forest, out: Optional[Schedule] = None, stream=None) -> Schedule:
    """jdb_schedule without a caller workspace: the scratch is a fixed array inside the library.

    For callers that cannot allocate device memory.  Limited to STATIC_MAX_NODES nodes; calls on one device
    share the scratch, so keep them on one stream.
    """
    out = alloc_schedule(forest.n_nodes, forest.child_ptr.device) if out is None else out
    cf, cs = forest.c(), out.c()
    st = lib().jdb_schedule_static(C.byref(cf), C.byref(cs), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_schedule_static")
    out.n_levels, out.n_leaves, out.n_wide_levels = cs.n_levels, cs.n_leaves, cs.n_wide_levels
    return out


def jdb_pack_weights(W: torch.Tensor, U: torch.Tensor, b: torch.Tensor, precision: int, stream=None) -> torch.Tensor:
    H, D = U.shape[1], W.shape[1]
    assert W.shape == (4 * H, D) and U.shape == (4 * H, H) and b.shape == (4 * H,)
    W, U, b = (t.to(torch.float32).contiguous() for t in (W, U, b))
    nbytes = lib().jdb_packed_weights_bytes(D, H, precision)
    packed = _device_bytes(nbytes, W.device)
    st = lib().jdb_pack_weights(_ptr(W), _ptr(U), _ptr(b), D, H, precision, _ptr(packed), packed.numel(), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_pack_weights")
    return packed


def forward_workspace(forest: Forest, sched: Schedule, D: int, H: int, precision: int) -> torch.Tensor:
    bound = forest.n_nodes - sched.n_leaves if sched.n_leaves >= 0 else forest.n_nodes
    return _device_bytes(lib().jdb_forward_workspace_bytes(forest.n_nodes, bound, D, H, precision),
                         forest.child_ptr.device)


def jdb_treelstm_forward(forest: Forest, sched: Schedule, x: torch.Tensor, packed: torch.Tensor, D: int, H: int,
                         precision: int, mode: int = MODE_AUTO, h: Optional[torch.Tensor] = None,
                         c: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None, stream=None,
                         barrier_timeout_ns: int = 0, prof_events=None,
                         trace: Optional[torch.Tensor] = None, flags: int = 0, tuning: int = 0):
    """h, c [n_nodes, H] fp32 of every node; x is fp32 or bfloat16 [n_nodes, >= D] with row stride x.stride(0)."""
    dev = forest.child_ptr.device
    n = forest.n_nodes
    if h is None:
        h = torch.empty((max(n, 1), H), dtype=torch.float32, device=dev)
    if c is None:
        c = torch.empty((max(n, 1), H), dtype=torch.float32, device=dev)
    if x.dtype == torch.bfloat16:
        x_dtype = BF16
    elif x.dtype == torch.float32:
        x_dtype = FP32
    else:
        raise TypeError("x must be float32 or bfloat16")
    assert x.stride(1) == 1 and h.stride(1) == 1 and c.stride(1) == 1 and h.stride(0) == c.stride(0)
    ws = forward_workspace(forest, sched, D, H, precision) if ws is None else ws
    cf, cs = forest.c(), sched.c()
    opts = COpts(precision, mode, flags, tuning, barrier_timeout_ns)
    if prof_events is not None:  # three torch.cuda.Event(enable_timing=True): begin, projection done, levels done
        for ev in prof_events:
            if ev.cuda_event == 0:
                ev.record()      # torch creates the CUDA event lazily, on first record
        opts.ev_begin, opts.ev_xproj_done, opts.ev_levels_done = (ev.cuda_event for ev in prof_events)
    if trace is not None:  # int64 cuda tensor receiving the level trace of the cooperative level loop
        opts.trace, opts.trace_cap = trace.data_ptr(), trace.numel()
    st = lib().jdb_treelstm_forward(C.byref(cf), C.byref(cs), _ptr(x), x_dtype, x.stride(0), _ptr(packed), D, H,
                                    _ptr(h), _ptr(c), h.stride(0), C.byref(opts), _ptr(ws), ws.numel(), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_treelstm_forward")
    return h[:n], c[:n]


def jdb_sched_status(sched: Schedule, stream=None):
    """Synchronise and raise what the device recorded (malformed forest, timed-out wait); returns (n_levels, n_leaves)."""
    cs = sched.c()
    nl, nv = C.c_int32(0), C.c_int32(0)
    st = lib().jdb_sched_status(C.byref(cs), C.byref(nl), C.byref(nv), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_sched_status")
    return nl.value, nv.value


def jdb_launch_counts(forest: Forest, sched: Schedule, ws: Optional[torch.Tensor] = None, stream=None):
    """(cells_unbatched, cells_batched, ops_unbatched, ops_batched, n_levels): Section 3's launch counts of the forest."""
    ws = _device_bytes(lib().jdb_launch_counts_workspace_bytes(forest.n_nodes), forest.child_ptr.device) if ws is None else ws
    cf, cs, out = forest.c(), sched.c(), CLaunchStats()
    st = lib().jdb_launch_counts(C.byref(cf), C.byref(cs), C.byref(out), _ptr(ws), ws.numel(), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_launch_counts")
    return out.cells_unbatched, out.cells_batched, out.ops_unbatched, out.ops_batched, out.n_levels


def jdb_relatedness_head(h: torch.Tensor, left: torch.Tensor, right: torch.Tensor, Wx: torch.Tensor, Wp: torch.Tensor,
                         bh: torch.Tensor, Wq: torch.Tensor, bq: torch.Tensor, stream=None, want_p: bool = True):
    """(y [P], p [P, K]) for pairs of root states taken from h [n, >= H] (fp32, row stride h.stride(0))."""
    Hs, H = Wx.shape
    K = Wq.shape[0]
    P = int(left.numel())
    dev = h.device
    Wx, Wp, bh, Wq, bq = (t.to(torch.float32).contiguous() for t in (Wx, Wp, bh, Wq, bq))
    left, right = left.to(torch.int32).contiguous(), right.to(torch.int32).contiguous()
    y = torch.empty(max(P, 1), dtype=torch.float32, device=dev)
    p = torch.empty((max(P, 1), K), dtype=torch.float32, device=dev) if want_p else None
    bad = torch.zeros(1, dtype=torch.int32, device=dev)
    st = lib().jdb_relatedness_head(_ptr(h), h.stride(0), h.shape[0], _ptr(left), _ptr(right), P, _ptr(Wx), _ptr(Wp), _ptr(bh),
                                    _ptr(Wq), _ptr(bq), H, Hs, K, _ptr(y), _ptr(p), _ptr(bad), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_relatedness_head")
    return y[:P], (p[:P] if want_p else None), bad


def jdb_treelstm_backward(forest: Forest, sched: Schedule, x: torch.Tensor, W: torch.Tensor, U: torch.Tensor, b: torch.Tensor,
                          h: torch.Tensor, c: torch.Tensor, grad_h: torch.Tensor, grad_c: Optional[torch.Tensor] = None,
                          want_dx: bool = True, ws: Optional[torch.Tensor] = None, stream=None):
    """(dW [4H, D], dU [4H, H], db [4H], dx [n, D] or None) of L = <grad_h, h> + <grad_c, c>; fp32 device tensors.

    h and c are the forward outputs (row stride h.stride(0)); grad_h / grad_c are [n, >= H] with a common row stride.
    """
    H4, D = W.shape
    H = H4 // 4
    n = forest.n_nodes
    dev = x.device
    if x.dtype != torch.float32 or h.dtype != torch.float32 or c.dtype != torch.float32 or grad_h.dtype != torch.float32:
        raise ValueError("jdb_treelstm_backward computes in fp32: x, h, c and grad_h must be float32")
    if c.stride(0) != h.stride(0) or (grad_c is not None and grad_c.stride(0) != grad_h.stride(0)):
        raise ValueError("h and c (and grad_h and grad_c) must share a row stride")
    W, U, b = (t.to(torch.float32).contiguous() for t in (W, U, b))
    n_int = n - sched.n_leaves if sched.n_leaves >= 0 else n
    if ws is None:
        ws = _device_bytes(lib().jdb_treelstm_backward_workspace_bytes(n, forest.n_edges, n_int, H), dev)
    dW = torch.empty((4 * H, D), dtype=torch.float32, device=dev)
    dU = torch.empty((4 * H, H), dtype=torch.float32, device=dev)
    db = torch.empty(4 * H, dtype=torch.float32, device=dev)
    dx = torch.empty((max(n, 1), D), dtype=torch.float32, device=dev) if want_dx else None
    cf, cs = forest.c(), sched.c()
    st = lib().jdb_treelstm_backward(C.byref(cf), C.byref(cs), _ptr(x), x.stride(0) if n > 0 else D, _ptr(W), _ptr(U), _ptr(b), D, H,
                                     _ptr(h), _ptr(c), h.stride(0) if n > 0 else H, _ptr(grad_h), _ptr(grad_c),
                                     grad_h.stride(0) if n > 0 else H, _ptr(dW), _ptr(dU), _ptr(db), _ptr(dx), D, _ptr(ws), ws.numel(),
                                     _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_treelstm_backward")
    return dW, dU, db, (dx[:n] if want_dx else None)


class CPlan(C.Structure):
    _fields_ = [("perm", C.c_void_p), ("slot_ptr", C.c_void_p), ("slot_depth", C.c_void_p), ("slot_key", C.c_void_p),
                ("n_slots", C.c_int32), ("bad_key", C.c_int32)]


class CCell(C.Structure):
    _fields_ = [("kind", C.c_int32), ("arity", C.c_int32), ("W", C.c_void_p), ("U", C.c_void_p), ("b", C.c_void_p)]


@dataclass
class Plan:
    perm: torch.Tensor        # int32 [n_nodes]: node ids by (depth, key, id)
    slot_ptr: torch.Tensor    # int32, entries 0..n_slots valid
    slot_depth: torch.Tensor
    slot_key: torch.Tensor
    n_slots: int = 0

    def c(self) -> CPlan:
        return CPlan(self.perm.data_ptr(), self.slot_ptr.data_ptr(), self.slot_depth.data_ptr(), self.slot_key.data_ptr(),
                     self.n_slots, 0)


def jdb_batch_plan(forest: Forest, sched: Schedule, key: torch.Tensor, n_keys: int, stream=None) -> Plan:
    """The table of Section 4.2 for nodes of several kinds: slots by (depth, key), ids ascending inside a slot."""
    dev = forest.child_ptr.device
    n = max(forest.n_nodes, 1)
    mk = lambda k: torch.empty(k, dtype=torch.int32, device=dev)
    out = Plan(mk(n), mk(n + 1), mk(n), mk(n))
    key = key.to(torch.int32).contiguous()
    ws = _device_bytes(lib().jdb_batch_plan_workspace_bytes(forest.n_nodes), dev)
    cf, cs, cp = forest.c(), sched.c(), out.c()
    st = lib().jdb_batch_plan(C.byref(cf), C.byref(cs), _ptr(key), n_keys, C.byref(cp), _ptr(ws), ws.numel(), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_batch_plan")
    out.n_slots = cp.n_slots
    return out


def jdb_cells_forward(forest: Forest, plan: Plan, key: torch.Tensor, cells, x: torch.Tensor, D: int, H: int,
                      h: Optional[torch.Tensor] = None, c: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                      stream=None):
    """h, c [n_nodes, H] fp32 of a forest whose node v is a cell of kind cells[key[v]].

    cells: list of (kind, arity, W, U, b) with fp32 device tensors (kind CELL_CHILDSUM or CELL_NARY).
    """
    dev = forest.child_ptr.device
    n = max(forest.n_nodes, 1)
    h = torch.empty((n, H), dtype=torch.float32, device=dev) if h is None else h
    c = torch.empty((n, H), dtype=torch.float32, device=dev) if c is None else c
    key = key.to(torch.int32).contiguous()
    keep = [tuple(t.to(torch.float32).contiguous() for t in cell[2:5]) for cell in cells]   # alive until the call returns
    arr = (CCell * len(cells))(*[CCell(int(cell[0]), int(cell[1]), W.data_ptr(), U.data_ptr(), b.data_ptr())
                                 for cell, (W, U, b) in zip(cells, keep)])
    amax = max([int(cell[1]) for cell in cells if int(cell[0]) == CELL_NARY] + [0])
    if ws is None:
        ws = _device_bytes(lib().jdb_cells_forward_workspace_bytes(forest.n_nodes, forest.n_edges, H, amax, len(cells)), dev)
    cf, cp = forest.c(), plan.c()
    st = lib().jdb_cells_forward(C.byref(cf), C.byref(cp), _ptr(key), arr, len(cells), _ptr(x), x.stride(0) if forest.n_nodes else D,
                                 D, H, _ptr(h), _ptr(c), h.stride(0), _ptr(ws), ws.numel(), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_cells_forward")
    return h[:forest.n_nodes], c[:forest.n_nodes]


def jdb_debug_report(sched: Schedule, stream=None):
    """(check, value, bound, where) recorded by a forward run with FLAG_DEBUG_CHECKS; check 0 means none failed."""
    cs = sched.c()
    out = (C.c_int32 * 4)()
    st = lib().jdb_debug_report(C.byref(cs), C.byref(out), _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_debug_report")
    return tuple(out)


class StepPlan:
    """One analysis + forward step with every argument marshalled ahead of time.

    For microsecond-scale forests the Python side of a call costs more than the kernels; the plan keeps the
    ctypes structures alive so that run() is two bare C calls (jdb_schedule_async, then jdb_treelstm_forward
    with JDB_FLAG_NO_SYNC when the level loop can run from the device-side level count).  Errors recorded on
    the device are raised by status(), which synchronises.
    """

    def __init__(self, forest: Forest, sched: Schedule, sws: torch.Tensor, x: torch.Tensor, packed: torch.Tensor,
                 D: int, H: int, precision: int, h: torch.Tensor, c: torch.Tensor, fws: torch.Tensor,
                 mode: int = MODE_AUTO, stream=None, async_schedule: bool = True):
        self.keep = (forest, sched, sws, x, packed, h, c, fws)
        self.sched = sched
        self.cf, self.cs = forest.c(), sched.c()
        self.cs.n_levels, self.cs.n_leaves, self.cs.n_wide_levels = -1, -1, -1
        self.opts = COpts(precision, mode, FLAG_NO_SYNC if async_schedule else 0, 0, 0, None, None, None, None, 0)
        self.stream = _stream(stream)
        self.async_schedule = async_schedule
        L = lib()
        self._sched_fn = L.jdb_schedule_async if async_schedule else L.jdb_schedule
        self._fwd_fn = L.jdb_treelstm_forward
        x_dtype = BF16 if x.dtype == torch.bfloat16 else FP32
        self._sched_args = (C.byref(self.cf), C.byref(self.cs), _ptr(sws), sws.numel(), self.stream)
        self._fwd_args = (C.byref(self.cf), C.byref(self.cs), _ptr(x), x_dtype, x.stride(0), _ptr(packed), D, H, _ptr(h),
                          _ptr(c), h.stride(0), C.byref(self.opts), _ptr(fws), fws.numel(), self.stream)

    def set_events(self, events):
        if events is None:
            self.opts.ev_begin = self.opts.ev_xproj_done = self.opts.ev_levels_done = None
            return
        for ev in events:
            if ev.cuda_event == 0:
                ev.record()
        self.opts.ev_begin, self.opts.ev_xproj_done, self.opts.ev_levels_done = (ev.cuda_event for ev in events)

    def run(self):
        st = self._sched_fn(*self._sched_args)
        if st != OK:
            raise JdbError(st, "jdb_schedule")
        st = self._fwd_fn(*self._fwd_args)
        if st != OK:
            raise JdbError(st, "jdb_treelstm_forward")

    def status(self):
        return jdb_sched_status(self.sched)


def forward_host_workspace(n_nodes: int, n_edges: int, D: int, H: int, precision: int, x_dtype: int,
                           device="cuda") -> torch.Tensor:
    return _device_bytes(lib().jdb_forward_host_workspace_bytes(n_nodes, n_edges, D, H, precision, x_dtype), device)


def jdb_treelstm_forward_host(child_ptr: torch.Tensor, child_idx: torch.Tensor, x: torch.Tensor, packed: torch.Tensor,
                              D: int, H: int, precision: int, h: torch.Tensor, c: torch.Tensor, dev_ws: torch.Tensor,
                              stream=None, flags: int = 0) -> int:
    """Host tensors in (CSR int32, x dense), host tensors out (h, c dense fp32).  Returns n_levels."""
    n, e = int(child_ptr.numel() - 1), int(child_idx.numel())
    for t in (child_ptr, child_idx, x, h, c):
        assert not t.is_cuda and t.is_contiguous()
    x_dtype = BF16 if x.dtype == torch.bfloat16 else FP32
    opts = COpts(precision, MODE_AUTO, flags, 0, 0, None, None, None, None, 0)
    nl = C.c_int32(0)
    st = lib().jdb_treelstm_forward_host(_ptr(child_ptr), _ptr(child_idx), n, e, _ptr(x), x_dtype, _ptr(packed), D, H,
                                         _ptr(h), _ptr(c), C.byref(opts), _ptr(dev_ws), dev_ws.numel(), C.byref(nl),
                                         _stream(stream))
    if st != OK:
        raise JdbError(st, "jdb_treelstm_forward_host")
    return nl.value


class Online:
    """Requests arriving one after the other: every request (a forest in host tensors) takes the next of `slots` slots, each
    with its own stream and device scratch, so new requests are copied and analysed while earlier ones execute.

    submit() returns a ticket; wait(ticket) returns that request's level count (its h and c host tensors are then
    filled) or raises its error.  The host tensors of a request must stay alive until it has been waited for.
    """

    def __init__(self, slots: int, max_nodes: int, max_edges: int, packed: torch.Tensor, D: int, H: int, precision: int,
                 x_dtype: int, device="cuda", flags: int = 0):
        self.D, self.H, self.x_dtype = D, H, x_dtype
        self.packed = packed
        self.ws = _device_bytes(lib().jdb_online_workspace_bytes(slots, max_nodes, max_edges, D, H, precision, x_dtype), device)
        opts = COpts(precision, MODE_AUTO, flags, 0, 0, None, None, None, None, 0)
        self.handle = C.c_void_p(None)
        st = lib().jdb_online_create(C.byref(self.handle), slots, max_nodes, max_edges, _ptr(packed), D, H, C.byref(opts), x_dtype,
                                     _ptr(self.ws), self.ws.numel())
        if st != OK:
            raise JdbError(st, "jdb_online_create")
        self._alive = {}

    def submit(self, child_ptr: torch.Tensor, child_idx: torch.Tensor, x: torch.Tensor, h: torch.Tensor, c: torch.Tensor) -> int:
        for t in (child_ptr, child_idx, x, h, c):
            assert not t.is_cuda and t.is_contiguous()
        assert (BF16 if x.dtype == torch.bfloat16 else FP32) == self.x_dtype
        n, e = int(child_ptr.numel() - 1), int(child_idx.numel())
        ticket = C.c_int64(-1)
        st = lib().jdb_online_submit(self.handle, _ptr(child_ptr), _ptr(child_idx), n, e, _ptr(x), _ptr(h), _ptr(c), C.byref(ticket))
        if st != OK:
            raise JdbError(st, "jdb_online_submit")
        self._alive[ticket.value] = (child_ptr, child_idx, x, h, c)
        return ticket.value

    def wait(self, ticket: int) -> int:
        nl = C.c_int32(0)
        st = lib().jdb_online_wait(self.handle, ticket, C.byref(nl))
        self._alive.pop(ticket, None)
        if st != OK:
            raise JdbError(st, "jdb_online_wait")
        return nl.value

    def close(self):
        if self.handle:
            lib().jdb_online_destroy(self.handle)
            self.handle = C.c_void_p(None)
            self._alive.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
