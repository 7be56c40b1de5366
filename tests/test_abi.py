"""The C-ABI library loads and exports every entry point that include/tsq.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2511_04002_b200 import binding as B
from paper_2511_04002_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_entry_points():
    text = open(os.path.join(ROOT, "include", "tsq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)                  # declarations only, not prose
    return sorted(set(re.findall(r"\b(tsq_[a-z_0-9]+)\s*\(", text)))


def test_header_and_binding_agree():
    names = declared_entry_points()
    assert "tsq_plan" in names and "tsq_encode" in names and "tsq_decode" in names
    assert sorted(B.EXPORTS) == names


def test_library_exports_every_declared_symbol():
    path = lib_build.build()
    lib = ctypes.CDLL(path)
    for name in declared_entry_points():
        assert hasattr(lib, name), name
    # calls that touch no GPU
    lib.tsq_status_string.restype = ctypes.c_char_p
    assert lib.tsq_status_string(0) == b"ok"
    assert lib.tsq_status_string(7) == b"device-side wait timed out"
    lib.tsq_kernel_launch_count.restype = ctypes.c_uint64
    assert lib.tsq_kernel_launch_count() == 0 or lib.tsq_kernel_launch_count() > 0


def test_plan_argument_errors_need_no_gpu():
    L = B.lib()
    h = ctypes.c_void_p()
    bits = (ctypes.c_int32 * 3)(2, 4, 8)
    bad = (ctypes.c_int32 * 2)(4, 4)
    assert L.tsq_plan(None, 0, 0, 256, 4, 6.0, bits, 3, 0.2, 0) == 1
    assert L.tsq_plan(ctypes.byref(h), 0, 5, 256, 4, 6.0, bits, 3, 0.2, 0) == 1            # dtype
    assert L.tsq_plan_variant(ctypes.byref(h), 0, 0, 256, 4, 6.0, bits, 3, 0.2, 0, 2) == 1  # variant
    assert L.tsq_plan_variant(ctypes.byref(h), 0, 0, 256, 4, 6.0, bits, 3, 0.2, 0, -1) == 1
    assert L.tsq_plan(ctypes.byref(h), 0, 0, 256, 4, 6.0, bad, 2, 0.2, 0) == 1             # not increasing
    assert L.tsq_plan(ctypes.byref(h), 0, 0, 100, 4, 6.0, bits, 3, 0.2, 0) == 2            # hidden % 8
    assert L.tsq_plan(ctypes.byref(h), 0, 0, 256, 4, float("nan"), bits, 3, 0.2, 0) == 1   # tau
    assert L.tsq_plan(ctypes.byref(h), 0, 0, 65536, 1 << 20, 6.0, bits, 3, 0.2, 0) == 1    # tokens * hidden >= 2^32
    assert not h.value
