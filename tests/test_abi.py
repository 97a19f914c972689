"""The C ABI library loads and exports every function include/asynclm.h declares (no GPU calls)."""
import ctypes
import os
import re

from paper_2412_07017_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "asynclm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(asynclm_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported():
    lib = B.load()
    names = declared_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), n
    assert set(B.EXPORTS) == set(names)


def test_version_and_strerror():
    lib = B.load()
    assert lib.asynclm_version() >= 100
    assert B.strerror(0) == "ok"
    for code in range(-8, 0):
        assert B.strerror(code) not in ("ok", "unknown status")
    assert B.strerror(-99) == "unknown status"


def test_struct_sizes_match_header_layout():
    assert ctypes.sizeof(B.CShape) == 32
    assert ctypes.sizeof(B.CPlanOptions) == 16
    assert ctypes.sizeof(B.CPlanInfo) == 12 * 4 + 3 * 8
    assert B.ITEM_DTYPE.itemsize == 32
