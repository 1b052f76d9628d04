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
