"""CPU-only: the C-ABI library builds, loads without a GPU and exports every declared symbol."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for h in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", h)).read()
        names += re.findall(r"PRISM_API\s+[\w\s\*]+?\b(prism_\w+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2510_15620_b200 import _build
    path = _build.build()
    L = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 16, names
    for n in names:
        assert hasattr(L, n), f"{n} declared in include/ but not exported"


def test_status_strings_and_null_handling():
    import paper_2510_15620_b200 as P
    assert P.status_str(0) == "PRISM_OK"
    assert P.status_str(-6) == "PRISM_ERR_TIMEOUT"
    assert P.status_str(-123) == "PRISM_ERR_UNKNOWN"
    L = P.lib()
    L.prism_destroy(None)                                  # allowed
    assert L.prism_last_error(None) == b""
    assert L.prism_create(None, None, None) == -1          # INVALID_ARG, no device touched


def test_record_layout_matches_header():
    from paper_2510_15620_b200 import ops
    assert ops.RECORD_BYTES == 80


def test_missing_library_fails_loudly(monkeypatch):
    import paper_2510_15620_b200.binding as B
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", "/nonexistent/libprism.so")
    with pytest.raises(ImportError):
        B.lib()


def test_route_entry_points_refuse_bad_arguments_before_any_launch():
    """An unknown mode, a FIXED_KEEP count below 1 or a ddof other than 0/1 would make the routing kernel write in
    front of the caller's buffers; both one-step entry points return INVALID_ARG first (no device is touched: this
    test runs without one, and the pointers are never followed)."""
    import paper_2510_15620_b200 as P
    L = P.lib()
    buf = (ctypes.c_int32 * 16)()
    fbuf = (ctypes.c_float * 16)()
    p, fp = ctypes.cast(buf, ctypes.c_void_p), ctypes.cast(fbuf, ctypes.c_void_p)

    def call(fn, n=4, mode=2, keep=0, clusters=3, ddof=0):
        fn.restype = ctypes.c_int
        return fn(fp, p, p, ctypes.c_int32(n), ctypes.c_int32(mode), ctypes.c_int32(keep), ctypes.c_double(0.5),
                  ctypes.c_int32(clusters), ctypes.c_int32(ddof), ctypes.c_int32(1), ctypes.c_int32(0), ctypes.c_int32(1),
                  p, p, p, p, p, fp, None, None)

    for fn in (L.prism_op_route, L.prism_op_route_static):
        assert call(fn, mode=3) == -1
        assert call(fn, mode=-1) == -1
        assert call(fn, mode=1, keep=0) == -1
        assert call(fn, mode=1, keep=-5) == -1
        assert call(fn, ddof=2) == -1
        assert call(fn, clusters=1) == -1
        assert call(fn, n=-1) == -1
    assert call(L.prism_op_route_static, n=1025) == -2        # beyond the built-in scratch: SHAPE_LIMIT
