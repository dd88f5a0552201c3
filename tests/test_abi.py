"""The C-ABI library loads and exports every function that include/taurus.h declares (no compute calls)."""
import os
import re

import paper_2607_17374_b200 as tb
from paper_2607_17374_b200 import build as tb_build
from paper_2607_17374_b200.binding import EXPORTS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "taurus.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(taurus_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    tb_build.build()          # nvcc cross-compiles without a GPU; no-op when up to date
    lib = tb.load_library()
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(EXPORTS) == names


def test_error_strings_without_a_device():
    lib = tb.load_library()
    assert lib.taurus_strerror(0) == b"ok"
    for code in tb.ERROR_CODES.values():
        assert lib.taurus_strerror(code) not in (b"", b"unknown error")
    assert lib.taurus_strerror(-99) == b"unknown error"


def test_missing_library_fails_loudly(monkeypatch):
    import paper_2607_17374_b200.binding as b
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "library_path", lambda: "/nonexistent/libtaurus.so")
    try:
        b.load_library()
    except RuntimeError as e:
        assert "no CPU fallback" in str(e)
    else:
        raise AssertionError("expected a RuntimeError")


def test_noalloc_entry_point_checks_its_sizes_before_touching_the_device():
    """Size and pointer checks of the allocation-free entry point come before its first CUDA call, so they can be
    exercised without a GPU."""
    assert tb.completion_counts_noalloc(0, 0, 1, 1, None, 1, 1) == tb.ERROR_CODES["INVALID_ARG"]
    assert tb.completion_counts_noalloc(10, -1, 1, 1, None, 1, 1) == tb.ERROR_CODES["INVALID_ARG"]
    assert tb.completion_counts_noalloc(10, 5, 1, None, None, 1, 1) == tb.ERROR_CODES["INVALID_ARG"]     # edges but no destinations
    assert tb.completion_counts_noalloc(10, 0, None, None, None, 1, 1) == tb.ERROR_CODES["INVALID_ARG"]
    assert tb.completion_counts_noalloc(tb.NOALLOC_MAX_VERTICES + 1, 0, 1, None, None, 1, 1) == tb.ERROR_CODES["UNSUPPORTED"]
