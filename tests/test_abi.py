"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and every validation path that precedes the first CUDA call returns its code."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def rs():
    from paper_2507_17307_b200 import build
    build.build_library()
    import paper_2507_17307_b200 as rs
    return rs


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(rstitch_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(rs):
    L = ctypes.CDLL(rs.library_path())
    names = declared_symbols()
    assert {"rstitch_route", "rstitch_route_ex", "rstitch_create", "rstitch_destroy",
            "rstitch_workspace_bytes", "rstitch_compact", "rstitch_last_status",
            "rstitch_status_string"} <= names
    for n in sorted(names):
        assert hasattr(L, n), n
    from paper_2507_17307_b200 import binding
    assert set(binding.EXPORTS) <= names


def test_status_strings(rs):
    seen = {rs.status_string(s) for s in range(-6, 1)}
    assert len(seen) == 7 and "ok" in seen
    assert rs.status_string(-99) == "unknown status"


def test_workspace_bytes(rs):
    assert rs.workspace_bytes(1, 1536, 151936) > 0
    assert rs.workspace_bytes(544, 5120, 152064) >= rs.workspace_bytes(1, 1536, 151936)
    assert rs.workspace_bytes(1, 1537, 100) == 0      # d % 8 != 0
    assert rs.workspace_bytes(1, 0, 100) == 0
    assert rs.workspace_bytes(1, 8, 1) == 0           # V < 2
    assert rs.workspace_bytes(-1, 8, 16) == 0


def test_validation_before_any_cuda_call(rs):
    L = rs.lib()
    one = ctypes.c_int32(0)
    p = ctypes.addressof(one)
    # shape errors of the basic form
    assert L.rstitch_route(p, p, 1, 12, 100, 0.5, p, p, p, p, p) == -3
    assert L.rstitch_route(p, p, 1, 4, 100, 0.5, p, p, p, p, p) == -3
    assert L.rstitch_route(p, p, 1, 8, 1, 0.5, p, p, p, p, p) == -3
    assert L.rstitch_route(p, p, -1, 8, 16, 0.5, p, p, p, p, p) == -1
    # extended form without a handle, and without arguments
    assert L.rstitch_route_ex(None, None, None) == -1
    # compaction
    assert L.rstitch_compact(p, -1, p, p, None) == -1
    assert L.rstitch_compact(None, 4, p, p, None) == -1
    assert L.rstitch_compact(p, 4, p, None, None) == -1
    # handle creation
    assert L.rstitch_create(None, 1, 8, 16) == -1
    h = ctypes.c_void_p()
    assert L.rstitch_create(ctypes.byref(h), 1, 7, 16) == -3
    assert L.rstitch_destroy(None) == 0
    assert L.rstitch_last_status(None, None) == -1
    assert L.rstitch_route_host(None, p, p, 1, 8, 16, 0.5, p, p, p, p, p, None) == -1


def test_alg1_validation_before_any_cuda_call(rs):
    import ctypes as C
    from paper_2507_17307_b200.binding import _Alg1State, LatencyModel
    L = rs.lib()
    one = C.c_int32(0)
    p = C.addressof(one)
    st = _Alg1State()
    lat = LatencyModel(0.0, 0.0, 0.0, 1.0)
    assert L.rstitch_alg1_init(C.byref(st), 4, p, None) == -1            # state arrays missing
    for k, _ in _Alg1State._fields_[:-1]:
        setattr(st, k, p)
    st.y_cap = 0
    assert L.rstitch_alg1_init(C.byref(st), 4, p, None) == -1            # no room for tokens
    st.y_cap = 8
    assert L.rstitch_alg1_init(C.byref(st), -1, p, None) == -1
    assert L.rstitch_alg1_init(C.byref(st), 4, None, None) == -1
    assert L.rstitch_alg1_init(C.byref(st), 0, None, None) == 0          # empty batch: nothing to launch
    assert L.rstitch_alg1_plan(C.byref(st), 4, 2, 8, C.byref(lat), p, p, p, p, p, None) == -1     # model id
    assert L.rstitch_alg1_plan(C.byref(st), 4, 0, -1, C.byref(lat), p, p, p, p, p, None) == -1    # T_max
    assert L.rstitch_alg1_plan(C.byref(st), 4, 0, 8, None, p, p, p, p, p, None) == -1
    assert L.rstitch_alg1_plan(C.byref(st), 4, 0, 8, C.byref(lat), None, p, p, p, p, None) == -1
    assert L.rstitch_alg1_plan(C.byref(st), 4, 0, 8, C.byref(LatencyModel(float("inf"), 0, 0, 0)), p, p, p, p, p,
                               None) == -1
    assert L.rstitch_alg1_commit(C.byref(st), 4, 0, p, None, None, p, p, 0, None) == -1
    assert L.rstitch_alg1_commit(C.byref(st), 4, 3, p, p, None, p, p, 0, None) == -1
    assert L.rstitch_alg1_commit(C.byref(st), 0, 0, None, p, None, None, None, 0, None) == 0
    assert L.rstitch_route_ex_host(None, None, None) == -1


def test_missing_library_fails_loudly(rs, monkeypatch):
    from paper_2507_17307_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/librstitch.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2507_17307_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in text.lower(), fn
    text = open(os.path.join(ROOT, "oracle", "rstitch_oracle.c")).read()
    assert "rstitch.h" not in text and "csrc" not in text
