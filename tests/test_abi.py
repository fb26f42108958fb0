"""Host-side checks that need no GPU: the library loads, exports every declared symbol, and
rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "spsyrk.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2608_09713_b200 import build
    return ctypes.CDLL(build.build_cuda())


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spsyrk_[a-z_]+)\s*\(", text)))


def test_header_declares_the_five_entry_points():
    names = declared_functions()
    for required in ("spsyrk_plan", "spsyrk_symbolic", "spsyrk_numeric", "spsyrk_mirror", "spsyrk_jaccard"):
        assert required in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in spsyrk.h but not exported"


def test_bounds_checked_build_exports_the_same_symbols():
    from paper_2608_09713_b200 import build
    checked = ctypes.CDLL(build.build_cuda(checked=True))
    for name in declared_functions():
        assert hasattr(checked, name), f"{name} is missing from the bounds-checked build"


def test_status_strings(lib):
    lib.spsyrk_status_string.restype = ctypes.c_char_p
    seen = {lib.spsyrk_status_string(i) for i in range(9)}
    assert len(seen) == 9 and lib.spsyrk_status_string(0) == b"ok"


def test_argument_errors_without_device(lib):
    sz = ctypes.c_size_t(0)
    i64 = ctypes.c_int64
    args = lambda m, n, nnz, dtype=0, mode=0, r0=0, r1=None: (
        None, i64(m), i64(n), i64(nnz), None, None, None, dtype, mode, i64(r0), i64(m if r1 is None else r1),
        None, ctypes.byref(sz), None)
    assert lib.spsyrk_plan(*args(10, 10, 20)) == 0 and sz.value > 0          # size query needs no device
    small = sz.value
    assert lib.spsyrk_plan(*args(1000, 10, 20000)) == 0 and sz.value > small
    assert lib.spsyrk_plan(*args(-1, 10, 20)) == 1
    assert lib.spsyrk_plan(*args(10, 10, 20, dtype=7)) == 1
    assert lib.spsyrk_plan(*args(10, 10, 20, mode=2)) == 1
    assert lib.spsyrk_plan(*args(10, 10, 20, r0=5, r1=4)) == 1
    assert lib.spsyrk_plan(*args(10, 10, 20, r1=11)) == 1
    assert lib.spsyrk_plan(*args(1 << 31, 10, 20)) == 4                       # overflow
    assert lib.spsyrk_plan(*args(10, 10, 1 << 31)) == 4
    assert lib.spsyrk_symbolic(None, None, None, None) == 1
    assert lib.spsyrk_numeric(None, None, None, None, None) == 1
    assert lib.spsyrk_plan_stats(None, None, None) == 1
    lib.spsyrk_destroy(None)                                                  # no-op
    assert lib.spsyrk_mirror(i64(10), i64(30), 0, None, None, None, None, None, None, None, None, ctypes.byref(sz), None) == 0
    assert sz.value > 0
    assert lib.spsyrk_mirror(i64(-1), i64(30), 0, None, None, None, None, None, None, None, None, ctypes.byref(sz), None) == 1
    assert lib.spsyrk_jaccard(i64(10), i64(5), i64(6), None, None, None, None, None, None) == 1
    panel = lambda m, k0, k1: lib.spsyrk_column_panel(i64(m), i64(30), 0, None, None, None, i64(k0), i64(k1), None, None, None,
                                                      None, None, ctypes.byref(sz), None)
    assert panel(10, 0, 5) == 0 and sz.value > 0
    assert panel(10, 5, 4) == 1 and panel(-1, 0, 5) == 1
    acc = lambda m, dt: lib.spsyrk_accumulate(i64(m), dt, i64(30), None, None, None, i64(20), None, None, None, None, None,
                                              None, None, None, ctypes.byref(sz), None)
    assert acc(10, 0) == 0 and sz.value > 0
    assert acc(-1, 0) == 1 and acc(10, 7) == 1
    perm = lambda m, n: lib.spsyrk_permute(i64(m), i64(n), i64(30), 0, None, None, None, None, None, None, None, None, None,
                                           ctypes.byref(sz), None)
    assert perm(10, 12) == 0 and sz.value > 0
    assert perm(-1, 12) == 1 and perm(1 << 31, 12) == 4
    assert lib.spsyrk_plan_partition(None, i64(4), None, None) == 1


def test_binding_mirrors_the_header():
    from paper_2608_09713_b200 import binding
    for name in declared_functions():
        assert hasattr(binding, name), f"binding lacks {name}"
