"""The C-ABI library loads without a GPU and exports what include/bls.h declares."""
import ctypes
import os
import re

import paper_2512_19342_b200 as bls
from paper_2512_19342_b200 import build as bls_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "bls.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bls_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    bls_build.build()
    lib = bls.lib()
    names = _declared()
    assert "bls_plan" in names and "bls_route" in names and "bls_lookup" in names and "bls_step" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(bls.EXPORTS) == names


def test_host_only_argument_checks():
    """Calls that never touch the GPU: sizes, argument validation, messages."""
    lib = bls.lib()
    assert lib.bls_strerror(0) == b"ok"

    class T(ctypes.Structure):
        _fields_ = [("w", ctypes.c_void_p), ("rows", ctypes.c_int64), ("dim", ctypes.c_int32), ("dt", ctypes.c_int32)]
    tabs = (T * 2)(T(256, 100, 16, 0), T(512, 50, 16, 0))
    n = ctypes.c_size_t(0)
    ok = lib.bls_plan_bytes(tabs, 2, 0, 2, 4, 2, ctypes.c_int64(64), ctypes.byref(n))
    assert ok == 0 and n.value > 0
    n1 = ctypes.c_size_t(0)
    lib.bls_plan_bytes(tabs, 2, 0, 2, 4, 3, ctypes.c_int64(64), ctypes.byref(n1))
    n0 = ctypes.c_size_t(0)
    lib.bls_plan_bytes(tabs, 2, 0, 2, 4, 1, ctypes.c_int64(64), ctypes.byref(n0))
    # ring memory grows linearly in k (one more slot per unit) ...
    assert n1.value - n.value == n.value - n0.value > 0
    # ... and does not depend on the table heights (Section V-F)
    tabs2 = (T * 2)(T(256, 100000, 16, 0), T(512, 5, 16, 0))
    n2 = ctypes.c_size_t(0)
    lib.bls_plan_bytes(tabs2, 2, 0, 2, 4, 2, ctypes.c_int64(64), ctypes.byref(n2))
    assert n2.value == n.value
    # one slot's output block is s*b*|tables| bytes per rank: dim 16 fp32 = 64 B vectors
    assert (n1.value - n.value) >= 2 * 4 * 2 * 64
    # rejected shapes
    assert lib.bls_plan_bytes(tabs, 2, 0, 33, 4, 2, ctypes.c_int64(64), ctypes.byref(n)) == bls.BLS_EINVAL
    assert lib.bls_plan_bytes(tabs, 2, 0, 2, 4, 16, ctypes.c_int64(64), ctypes.byref(n)) == bls.BLS_EINVAL
    bad = (T * 1)(T(256, 100, 24, 0))            # 96-byte rows are not supported
    assert lib.bls_plan_bytes(bad, 1, 0, 2, 4, 2, ctypes.c_int64(64), ctypes.byref(n)) == bls.BLS_EINVAL
