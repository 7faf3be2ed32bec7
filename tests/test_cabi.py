"""Host-only checks of the C-ABI library: it builds, loads without a GPU, and exports what jdb.h declares."""
import ctypes
import os
import re

from conftest import ROOT
from paper_1904_07421_b200 import build as jbuild
from paper_1904_07421_b200 import jdb


def declared_functions():
    text = open(os.path.join(ROOT, "include", "jdb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(jdb_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    jbuild.build()
    assert os.path.exists(jdb.LIB_PATH)
    raw = ctypes.CDLL(jdb.LIB_PATH)
    names = declared_functions()
    assert len(names) >= 13
    for name in names:
        assert hasattr(raw, name), f"{name} declared in jdb.h but not exported"
    assert sorted(jdb.EXPORTS) == names


def test_host_only_queries():
    L = jdb.lib()
    assert L.jdb_status_string(jdb.OK) == b"ok"
    for code in range(8):
        assert len(L.jdb_status_string(code)) > 0
    small = L.jdb_schedule_workspace_bytes(1000, 999)
    big = L.jdb_schedule_workspace_bytes(1_600_000, 1_530_000)
    assert 0 < small < big
    assert big >= 4 * 4 * 1_600_000
    p32 = L.jdb_packed_weights_bytes(300, 150, jdb.FP32)
    assert p32 >= (300 + 150) * 600 * 4
    assert L.jdb_packed_weights_bytes(0, 150, jdb.FP32) == 0
    fw = L.jdb_forward_workspace_bytes(1000, 400, 300, 150, jdb.FP32)
    assert fw >= 400 * 600 * 4
    hw = L.jdb_forward_host_workspace_bytes(1000, 999, 300, 150, jdb.FP32, jdb.FP32)
    assert hw > fw + 2 * 1000 * 150 * 4
    # the entry points added beside the forward: sizes grow with what they hold, bad sizes give 0
    bw = L.jdb_treelstm_backward_workspace_bytes(1000, 999, 400, 150)
    assert bw >= (1000 * 4 * 150 + 2 * 1000 * 150 + 999 * 150) * 4 and L.jdb_treelstm_backward_workspace_bytes(-1, 0, 0, 150) == 0
    assert L.jdb_batch_plan_workspace_bytes(100000) >= 3 * 100000 * 4
    cw2, cw8 = (L.jdb_cells_forward_workspace_bytes(1000, 999, 150, a, 2) for a in (2, 8))
    assert 1000 * 4 * 150 * 4 < cw2 < cw8
    assert L.jdb_online_workspace_bytes(3, 1000, 999, 300, 150, jdb.FP32, jdb.FP32) >= 3 * hw
    assert L.jdb_online_workspace_bytes(0, 1000, 999, 300, 150, jdb.FP32, jdb.FP32) == 0
    # the host object of the online entry refuses bad arguments before it touches the device
    handle = ctypes.c_void_p(None)
    opts = jdb.COpts(jdb.FP32, jdb.MODE_AUTO, 0, 0, 0, None, None, None, None, 0)
    assert L.jdb_online_create(ctypes.byref(handle), 0, 10, 9, None, 4, 4, ctypes.byref(opts), jdb.FP32, None, 0) == jdb.ERR_INVALID_ARG
    assert not handle.value
    assert L.jdb_online_destroy(None) == jdb.OK


def L_places(n):
    return jdb.lib().jdb_launch_counts_workspace_bytes(n)


def test_struct_layouts_match_header():
    # field order and widths as declared in jdb.h (LP64)
    assert ctypes.sizeof(jdb.CForest) == 24
    assert ctypes.sizeof(jdb.CSched) == 48
    assert ctypes.sizeof(jdb.COpts) == 64
    assert ctypes.sizeof(jdb.CLaunchStats) == 40
    assert ctypes.sizeof(jdb.CPlan) == 40       # four pointers, two int32
    assert ctypes.sizeof(jdb.CCell) == 32       # two int32, three pointers
    assert L_places(1) >= 1024 * 8 and L_places(100000) >= 2 * 100000 * 8
