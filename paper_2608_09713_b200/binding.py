"""ctypes binding of libspsyrk.so: argument marshalling only.

Every function mirrors a C entry point of ``include/spsyrk.h`` under the same name and takes
torch CUDA tensors (device memory and streams are PyTorch's; the arithmetic is all in the
library's kernels).  Importing this module loads the CUDA library and raises if it is missing:
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SPSYRK_LIBRARY selects another build of the same library (the bounds-checked one, libspsyrk_checked.so)
LIB_PATH = os.environ.get("SPSYRK_LIBRARY") or os.path.join(_HERE, "libspsyrk.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2608_09713_b200.build` "
        "(nvcc, sm_100a).  The library has no CPU fallback.")

_lib = ctypes.CDLL(LIB_PATH)

OK = 0
F64, F32, I32 = 0, 1, 2
TRIL, FULL = 0, 1
NCLASS = 8

_DTYPE_CODE = {torch.float64: F64, torch.float32: F32, torch.int32: I32}
_CODE_DTYPE = {v: k for k, v in _DTYPE_CODE.items()}

_i64, _vp, _int = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
_szp = ctypes.POINTER(ctypes.c_size_t)
_i64p = ctypes.POINTER(ctypes.c_int64)

_lib.spsyrk_plan.argtypes = [ctypes.POINTER(_vp), _i64, _i64, _i64, _vp, _vp, _vp, _int, _int, _i64, _i64, _vp, _szp, _vp]
_lib.spsyrk_plan_set_rows.argtypes = [_vp, _i64, _i64, _vp]
_lib.spsyrk_plan_set_block.argtypes = [_vp, _i64, _i64, _i64, _i64, _vp]
_lib.spsyrk_plan_set_block.restype = _int
_lib.spsyrk_symbolic.argtypes = [_vp, _vp, _i64p, _vp]
_lib.spsyrk_plan_set_jaccard.argtypes = [_vp, _vp]
_lib.spsyrk_plan_set_jaccard.restype = _int
_lib.spsyrk_plan_map_bytes.argtypes = [_vp, _szp]
_lib.spsyrk_plan_map_bytes.restype = _int
_lib.spsyrk_plan_lend_map.argtypes = [_vp, _vp, ctypes.c_size_t]
_lib.spsyrk_plan_lend_map.restype = _int
_lib.spsyrk_numeric.argtypes = [_vp, _vp, _vp, _vp, _vp]
_lib.spsyrk_numeric_rows.argtypes = [_vp, _i64, _i64, _vp, _vp, _vp, _vp]
_lib.spsyrk_numeric_rows.restype = _int
_lib.spsyrk_onepass_slots.argtypes = [_vp, _i64p, _vp]
_lib.spsyrk_onepass_slots.restype = _int
_lib.spsyrk_onepass_numeric.argtypes = [_vp, _vp, _vp, _vp, _i64p, _vp]
_lib.spsyrk_onepass_numeric.restype = _int
_lib.spsyrk_onepass_compact.argtypes = [_vp, _vp, _i64, _vp, _vp, _vp, _vp, _vp]
_lib.spsyrk_onepass_compact.restype = _int
_lib.spsyrk_onepass_row_begin.argtypes = [_vp, _vp, _vp]
_lib.spsyrk_onepass_row_begin.restype = _int
_lib.spsyrk_mirror.argtypes = [_i64, _i64, _int, _vp, _vp, _vp, _vp, _vp, _vp, _i64p, _vp, _szp, _vp]
_lib.spsyrk_column_panel.argtypes = [_i64, _i64, _int, _vp, _vp, _vp, _i64, _i64, _vp, _vp, _vp, _i64p, _vp, _szp, _vp]
_lib.spsyrk_accumulate.argtypes = [_i64, _int, _i64, _vp, _vp, _vp, _i64, _vp, _vp, _vp, _vp, _vp, _vp, _i64p, _vp, _szp, _vp]
_lib.spsyrk_permute.argtypes = [_i64, _i64, _i64, _int, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _szp, _vp]
_lib.spsyrk_plan_partition.argtypes = [_vp, _i64, _i64p, _vp]
_lib.spsyrk_host_release_cache.argtypes = []
_lib.spsyrk_mirror_rowptr_noalloc.argtypes = [_i64, _vp, _vp, _vp, _i64p, _vp]
_lib.spsyrk_mirror_rowptr_noalloc.restype = _int
_lib.spsyrk_symv.argtypes = [_i64, _i64, _int, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.spsyrk_symv.restype = _int
_lib.spsyrk_symm.argtypes = [_i64, _i64, _i64, _int, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.spsyrk_symm.restype = _int
_lib.spsyrk_jaccard.argtypes = [_i64, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.spsyrk_plan_stats.argtypes = [_vp, _i64p, _i64p]
_lib.spsyrk_plan_buffers.argtypes = [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp)]
_lib.spsyrk_destroy.argtypes = [_vp]
_lib.spsyrk_destroy.restype = None
_lib.spsyrk_status_string.argtypes = [_int]
_lib.spsyrk_status_string.restype = ctypes.c_char_p
_lib.spsyrk_host_tril.argtypes = [ctypes.POINTER(_vp), _i64, _i64, _i64, _vp, _vp, _vp, _int, _int, _vp, _i64p, _vp, _vp]
_lib.spsyrk_plan_enable_timing.argtypes = [_vp]
_lib.spsyrk_plan_timings.argtypes = [_vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float)]
_lib.spsyrk_mirror_enable_timing.argtypes = [_int]
_lib.spsyrk_mirror_enable_timing.restype = _int
_lib.spsyrk_mirror_timings.argtypes = [ctypes.POINTER(_int), ctypes.POINTER(ctypes.c_float)]
_lib.spsyrk_mirror_timings.restype = _int
_lib.spsyrk_launch_count.argtypes = []
_lib.spsyrk_launch_count.restype = ctypes.c_int64
for _name in ("spsyrk_plan_enable_timing", "spsyrk_plan_timings"):
    getattr(_lib, _name).restype = _int
for _name in ("spsyrk_plan", "spsyrk_plan_set_rows", "spsyrk_symbolic", "spsyrk_numeric", "spsyrk_mirror",
              "spsyrk_jaccard", "spsyrk_plan_stats", "spsyrk_plan_buffers", "spsyrk_host_tril", "spsyrk_column_panel",
              "spsyrk_accumulate", "spsyrk_permute", "spsyrk_plan_partition", "spsyrk_host_release_cache"):
    getattr(_lib, _name).restype = _int


class SpsyrkError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {spsyrk_status_string(status)} (status {status})")


def spsyrk_status_string(status: int) -> str:
    return _lib.spsyrk_status_string(status).decode()


def _check(status: int, where: str):
    if status != OK:
        raise SpsyrkError(status, where)


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dev_check(*tensors):
    for t in tensors:
        if t is not None and not (t.is_cuda and t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")


def _workspace(nbytes: int, device) -> torch.Tensor:
    # torch's caching allocator returns 512-byte aligned blocks
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


class Plan:
    """Owner of a spsyrk_plan_t and of the tensors it borrows (A and the workspace)."""

    def __init__(self, handle, keep, m, n, dtype, mode):
        self._h, self._keep = handle, keep
        self.m, self.n, self.dtype, self.mode = m, n, dtype, mode
        self.row_begin, self.row_end = keep["rows"]

    @property
    def rows(self):
        return self.row_end - self.row_begin

    def close(self):
        # at interpreter shutdown the module's globals may already be gone: the process exit frees the plan
        if self._h is not None and _lib is not None:
            _lib.spsyrk_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()


def spsyrk_plan_workspace_bytes(m, n, nnz, dtype=torch.float64, mode=TRIL) -> int:
    sz = ctypes.c_size_t(0)
    _check(_lib.spsyrk_plan(None, m, n, nnz, None, None, None, _DTYPE_CODE[dtype], mode, 0, m, None,
                            ctypes.byref(sz), None), "spsyrk_plan(size query)")
    return sz.value


def spsyrk_plan(m, n, rowptr, colidx, vals, mode=TRIL, row_begin=0, row_end=None, stream=None, workspace=None) -> Plan:
    _dev_check(rowptr, colidx, vals)
    assert rowptr.dtype == torch.int64 and colidx.dtype == torch.int32 and vals.dtype in _DTYPE_CODE
    row_end = m if row_end is None else row_end
    nnz = colidx.numel()
    code = _DTYPE_CODE[vals.dtype]
    sz = ctypes.c_size_t(0)
    _check(_lib.spsyrk_plan(None, m, n, nnz, None, None, None, code, mode, row_begin, row_end, None,
                            ctypes.byref(sz), None), "spsyrk_plan(size query)")
    ws = workspace if workspace is not None else _workspace(sz.value, rowptr.device)
    assert ws.numel() >= sz.value
    sz = ctypes.c_size_t(ws.numel())
    h = _vp()
    _check(_lib.spsyrk_plan(ctypes.byref(h), m, n, nnz, _p(rowptr), _p(colidx), _p(vals), code, mode, row_begin,
                            row_end, _p(ws), ctypes.byref(sz), _stream(stream)), "spsyrk_plan")
    return Plan(h, {"a": (rowptr, colidx, vals), "ws": ws, "rows": (row_begin, row_end)}, m, n, vals.dtype, mode)


def spsyrk_plan_set_rows(plan: Plan, row_begin: int, row_end: int, stream=None):
    _check(_lib.spsyrk_plan_set_rows(plan._h, row_begin, row_end, _stream(stream)), "spsyrk_plan_set_rows")
    plan.row_begin, plan.row_end = row_begin, row_end


def spsyrk_plan_set_block(plan: Plan, row_begin: int, row_end: int, col_begin: int, col_end: int, stream=None):
    """Restrict the plan to output rows [row_begin, row_end) and output columns [col_begin, col_end)."""
    _check(_lib.spsyrk_plan_set_block(plan._h, row_begin, row_end, col_begin, col_end, _stream(stream)),
           "spsyrk_plan_set_block")
    plan.row_begin, plan.row_end = row_begin, row_end


def spsyrk_plan_map_bytes(plan: Plan) -> int:
    sz = ctypes.c_size_t(0)
    _check(_lib.spsyrk_plan_map_bytes(plan._h, ctypes.byref(sz)), "spsyrk_plan_map_bytes")
    return sz.value


def spsyrk_plan_lend_map(plan: Plan, item_map: torch.Tensor | None):
    """Lend (or, with None, take back) the item map: a uint8 CUDA tensor of at least spsyrk_plan_map_bytes bytes."""
    if item_map is not None:
        _dev_check(item_map)
        assert item_map.dtype == torch.uint8
    _check(_lib.spsyrk_plan_lend_map(plan._h, _p(item_map), 0 if item_map is None else item_map.numel()),
           "spsyrk_plan_lend_map")
    plan._keep["map"] = item_map


def spsyrk_plan_set_jaccard(plan: Plan, jaccard: torch.Tensor | None):
    """From now on spsyrk_numeric also writes the Jaccard similarities into `jaccard` (float32 CUDA tensor with
    as many entries as the product; int32 plans only); None switches the fusion off."""
    if jaccard is not None:
        _dev_check(jaccard)
        assert jaccard.dtype == torch.float32
    _check(_lib.spsyrk_plan_set_jaccard(plan._h, _p(jaccard)), "spsyrk_plan_set_jaccard")
    plan._keep["jaccard"] = jaccard


def spsyrk_symbolic(plan: Plan, c_rowptr: torch.Tensor, stream=None) -> int:
    _dev_check(c_rowptr)
    assert c_rowptr.dtype == torch.int64 and c_rowptr.numel() >= plan.rows + 1
    nnz = ctypes.c_int64(0)
    _check(_lib.spsyrk_symbolic(plan._h, _p(c_rowptr), ctypes.byref(nnz), _stream(stream)), "spsyrk_symbolic")
    return nnz.value


def spsyrk_numeric(plan: Plan, c_rowptr, c_colidx, c_vals, stream=None):
    _dev_check(c_rowptr, c_colidx, c_vals)
    assert c_colidx.dtype == torch.int32 and c_vals.dtype == plan.dtype
    _check(_lib.spsyrk_numeric(plan._h, _p(c_rowptr), _p(c_colidx), _p(c_vals), _stream(stream)), "spsyrk_numeric")


def spsyrk_numeric_rows(plan: Plan, row_begin: int, row_end: int, c_rowptr, c_colidx, c_vals, stream=None):
    _dev_check(c_rowptr, c_colidx, c_vals)
    assert c_colidx.dtype == torch.int32 and c_vals.dtype == plan.dtype
    _check(_lib.spsyrk_numeric_rows(plan._h, int(row_begin), int(row_end), _p(c_rowptr), _p(c_colidx), _p(c_vals), _stream(stream)),
           "spsyrk_numeric_rows")


def spsyrk_onepass_slots(plan: Plan, stream=None) -> int:
    slots = ctypes.c_int64(0)
    _check(_lib.spsyrk_onepass_slots(plan._h, ctypes.byref(slots), _stream(stream)), "spsyrk_onepass_slots")
    return slots.value


def spsyrk_onepass_numeric(plan: Plan, slot_colidx, slot_vals, c_rowptr, stream=None) -> int:
    _dev_check(slot_colidx, slot_vals, c_rowptr)
    assert slot_colidx.dtype == torch.int32 and slot_vals.dtype == plan.dtype and c_rowptr.dtype == torch.int64
    nnz = ctypes.c_int64(0)
    _check(_lib.spsyrk_onepass_numeric(plan._h, _p(slot_colidx), _p(slot_vals), _p(c_rowptr), ctypes.byref(nnz), _stream(stream)),
           "spsyrk_onepass_numeric")
    return nnz.value


def spsyrk_onepass_row_begin(plan: Plan, row_begin, stream=None):
    _dev_check(row_begin)
    assert row_begin.dtype == torch.int64 and row_begin.numel() >= plan.rows + 1
    _check(_lib.spsyrk_onepass_row_begin(plan._h, _p(row_begin), _stream(stream)), "spsyrk_onepass_row_begin")
    return row_begin


def spsyrk_onepass_compact(plan: Plan, c_rowptr, nnz, slot_colidx, slot_vals, c_colidx, c_vals, stream=None):
    _dev_check(c_rowptr, slot_colidx, slot_vals, c_colidx, c_vals)
    _check(_lib.spsyrk_onepass_compact(plan._h, _p(c_rowptr), int(nnz), _p(slot_colidx), _p(slot_vals), _p(c_colidx), _p(c_vals),
                                       _stream(stream)), "spsyrk_onepass_compact")


def onepass_syrk(plan: Plan, stream=None, compact=True):
    """C_L through the one-pass mode: slots -> numeric into the slots -> compaction.  Returns (c_rowptr, c_colidx, c_vals);
    with compact=False the four-array form (row_begin, c_rowptr, slot_colidx, slot_vals): row r is
    slot_*[row_begin[r] : row_begin[r] + c_rowptr[r + 1] - c_rowptr[r]]."""
    dev = plan._keep["a"][0].device
    slots = spsyrk_onepass_slots(plan, stream)
    s_col = torch.empty(max(slots, 1), dtype=torch.int32, device=dev)
    s_val = torch.empty(max(slots, 1), dtype=plan.dtype, device=dev)
    c_rowptr = torch.empty(plan.rows + 1, dtype=torch.int64, device=dev)
    nnz = spsyrk_onepass_numeric(plan, s_col, s_val, c_rowptr, stream)
    if not compact:
        row_begin = spsyrk_onepass_row_begin(plan, torch.empty(plan.rows + 1, dtype=torch.int64, device=dev), stream)
        return row_begin, c_rowptr, s_col, s_val
    c_colidx = torch.empty(max(nnz, 1), dtype=torch.int32, device=dev)
    c_vals = torch.empty(max(nnz, 1), dtype=plan.dtype, device=dev)
    spsyrk_onepass_compact(plan, c_rowptr, nnz, s_col, s_val, c_colidx, c_vals, stream)
    return c_rowptr, c_colidx[:nnz], c_vals[:nnz]


def spsyrk_destroy(plan: Plan):
    plan.close()


def spsyrk_plan_stats(plan: Plan):
    work = ctypes.c_int64(0)
    cls = (ctypes.c_int64 * NCLASS)()
    _check(_lib.spsyrk_plan_stats(plan._h, ctypes.byref(work), cls), "spsyrk_plan_stats")
    return work.value, list(cls)


def spsyrk_plan_enable_timing(plan: Plan):
    _check(_lib.spsyrk_plan_enable_timing(plan._h), "spsyrk_plan_enable_timing")


def spsyrk_plan_timings(plan: Plan):
    """(symbolic_ms[8], numeric_ms[8]): device milliseconds per row class of the last calls."""
    sym = (ctypes.c_float * NCLASS)()
    num = (ctypes.c_float * NCLASS)()
    _check(_lib.spsyrk_plan_timings(plan._h, sym, num), "spsyrk_plan_timings")
    return list(sym), list(num)


def spsyrk_mirror_enable_timing(on: bool = True):
    _check(_lib.spsyrk_mirror_enable_timing(1 if on else 0), "spsyrk_mirror_enable_timing")


def spsyrk_mirror_timings():
    """Device milliseconds of the sorting passes of the last spsyrk_mirror fill on 8-byte values."""
    n = _int(0)
    ms = (ctypes.c_float * 4)()
    _check(_lib.spsyrk_mirror_timings(ctypes.byref(n), ms), "spsyrk_mirror_timings")
    return [float(ms[i]) for i in range(n.value)]


def spsyrk_launch_count() -> int:
    return int(_lib.spsyrk_launch_count())


def spsyrk_plan_buffers(plan: Plan):
    """Copies of the plan's column lists and work estimate as torch tensors: (colptr, at_row, at_val, work); the values
    are taken out of the plan's (row id, value) records."""
    ptrs = [_vp() for _ in range(4)]
    _check(_lib.spsyrk_plan_buffers(plan._h, *[ctypes.byref(p) for p in ptrs]), "spsyrk_plan_buffers")
    nnz = plan._keep["a"][1].numel()
    dev = plan._keep["a"][0].device

    def view(ptr, count, dtype):
        if count == 0:
            return torch.empty(0, dtype=dtype, device=dev)
        return torch.as_tensor(_DevArray(ptr.value, count, _TYPESTR[dtype]), device=dev).clone()

    torch.cuda.synchronize()
    # a record is (row id, [padding,] value): seen as 2 * nnz elements of the value type, the values are the odd ones
    at_val = view(ptrs[2], 2 * nnz, plan.dtype)[1::2].contiguous()
    return (view(ptrs[0], plan.n + 1, torch.int64), view(ptrs[1], nnz, torch.int32), at_val, view(ptrs[3], plan.rows, torch.int64))


_TYPESTR = {torch.int64: "<i8", torch.int32: "<i4", torch.float64: "<f8", torch.float32: "<f4"}


class _DevArray:
    """A device pointer dressed as a CUDA array so that torch can wrap it without copying."""

    def __init__(self, ptr, count, typestr):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (ptr, False), "version": 2}


def spsyrk_mirror_workspace_bytes(m, nnz_l, dtype) -> int:
    sz = ctypes.c_size_t(0)
    _check(_lib.spsyrk_mirror(m, nnz_l, _DTYPE_CODE[dtype], None, None, None, None, None, None, None, None,
                              ctypes.byref(sz), None), "spsyrk_mirror(size query)")
    return sz.value


def spsyrk_mirror(m, l_rowptr, l_colidx, l_vals, stream=None, workspace=None, out=None):
    """Returns (f_rowptr, f_colidx, f_vals) of F = C_L + C_L^T - D.  The outputs are allocated with torch
    unless `out` = (f_rowptr, f_colidx, f_vals) supplies buffers that are large enough."""
    _dev_check(l_rowptr, l_colidx, l_vals)
    nnz_l = l_colidx.numel()
    code = _DTYPE_CODE[l_vals.dtype]
    sz = ctypes.c_size_t(spsyrk_mirror_workspace_bytes(m, nnz_l, l_vals.dtype))
    ws = workspace if workspace is not None else _workspace(sz.value, l_rowptr.device)
    assert ws.numel() >= sz.value
    sz = ctypes.c_size_t(ws.numel())
    f_rowptr = out[0] if out is not None else torch.empty(m + 1, dtype=torch.int64, device=l_rowptr.device)
    nnz = ctypes.c_int64(0)
    st = _stream(stream)
    _check(_lib.spsyrk_mirror(m, nnz_l, code, _p(l_rowptr), _p(l_colidx), _p(l_vals), _p(f_rowptr), None, None,
                              ctypes.byref(nnz), _p(ws), ctypes.byref(sz), st), "spsyrk_mirror(sizes)")
    if out is not None:
        f_colidx, f_vals = out[1], out[2]
        assert f_colidx.numel() >= nnz.value and f_vals.numel() >= nnz.value and f_vals.dtype == l_vals.dtype
    else:
        f_colidx = torch.empty(max(nnz.value, 1), dtype=torch.int32, device=l_rowptr.device)
        f_vals = torch.empty(max(nnz.value, 1), dtype=l_vals.dtype, device=l_rowptr.device)
    _check(_lib.spsyrk_mirror(m, nnz_l, code, _p(l_rowptr), _p(l_colidx), _p(l_vals), _p(f_rowptr), _p(f_colidx),
                              _p(f_vals), ctypes.byref(nnz), _p(ws), ctypes.byref(sz), st), "spsyrk_mirror(fill)")
    return f_rowptr, f_colidx[:nnz.value], f_vals[:nnz.value]


def spsyrk_column_panel(m, rowptr, colidx, vals, k0, k1, stream=None, workspace=None):
    """Returns (p_rowptr, p_colidx, p_vals) of A(:, [k0, k1)), column ids unchanged."""
    _dev_check(rowptr, colidx, vals)
    nnz, code, dev = colidx.numel(), _DTYPE_CODE[vals.dtype], rowptr.device
    sz = ctypes.c_size_t(0)
    _check(_lib.spsyrk_column_panel(m, nnz, code, None, None, None, k0, k1, None, None, None, None, None,
                                    ctypes.byref(sz), None), "spsyrk_column_panel(size query)")
    ws = workspace if workspace is not None else _workspace(sz.value, dev)
    assert ws.numel() >= sz.value
    sz = ctypes.c_size_t(ws.numel())
    p_rowptr = torch.empty(m + 1, dtype=torch.int64, device=dev)
    out_nnz = ctypes.c_int64(0)
    st = _stream(stream)
    _check(_lib.spsyrk_column_panel(m, nnz, code, _p(rowptr), _p(colidx), _p(vals), k0, k1, _p(p_rowptr), None, None,
                                    ctypes.byref(out_nnz), _p(ws), ctypes.byref(sz), st), "spsyrk_column_panel(sizes)")
    p_colidx = torch.empty(max(out_nnz.value, 1), dtype=torch.int32, device=dev)
    p_vals = torch.empty(max(out_nnz.value, 1), dtype=vals.dtype, device=dev)
    _check(_lib.spsyrk_column_panel(m, nnz, code, _p(rowptr), _p(colidx), _p(vals), k0, k1, _p(p_rowptr), _p(p_colidx),
                                    _p(p_vals), ctypes.byref(out_nnz), _p(ws), ctypes.byref(sz), st), "spsyrk_column_panel(fill)")
    return p_rowptr, p_colidx[:out_nnz.value], p_vals[:out_nnz.value]


def spsyrk_accumulate(m, x_rowptr, x_colidx, x_vals, y_rowptr, y_colidx, y_vals, stream=None, workspace=None):
    """Returns (z_rowptr, z_colidx, z_vals) of Z = X + Y (union structure, x + y on shared entries)."""
    _dev_check(x_rowptr, x_colidx, x_vals, y_rowptr, y_colidx, y_vals)
    assert x_vals.dtype == y_vals.dtype
    nx, ny, code, dev = x_colidx.numel(), y_colidx.numel(), _DTYPE_CODE[x_vals.dtype], x_rowptr.device
    sz = ctypes.c_size_t(0)
    _check(_lib.spsyrk_accumulate(m, code, nx, None, None, None, ny, None, None, None, None, None, None, None, None,
                                  ctypes.byref(sz), None), "spsyrk_accumulate(size query)")
    ws = workspace if workspace is not None else _workspace(sz.value, dev)
    assert ws.numel() >= sz.value
    sz = ctypes.c_size_t(ws.numel())
    z_rowptr = torch.empty(m + 1, dtype=torch.int64, device=dev)
    nnz = ctypes.c_int64(0)
    st = _stream(stream)
    args = (m, code, nx, _p(x_rowptr), _p(x_colidx), _p(x_vals), ny, _p(y_rowptr), _p(y_colidx), _p(y_vals), _p(z_rowptr))
    _check(_lib.spsyrk_accumulate(*args, None, None, ctypes.byref(nnz), _p(ws), ctypes.byref(sz), st),
           "spsyrk_accumulate(sizes)")
    z_colidx = torch.empty(max(nnz.value, 1), dtype=torch.int32, device=dev)
    z_vals = torch.empty(max(nnz.value, 1), dtype=x_vals.dtype, device=dev)
    _check(_lib.spsyrk_accumulate(*args, _p(z_colidx), _p(z_vals), ctypes.byref(nnz), _p(ws), ctypes.byref(sz), st),
           "spsyrk_accumulate(fill)")
    return z_rowptr, z_colidx[:nnz.value], z_vals[:nnz.value]


def spsyrk_permute(m, n, rowptr, colidx, vals, rperm, cperm=None, stream=None, workspace=None):
    """Returns (b_rowptr, b_colidx, b_vals): row i of A at row rperm[i], column k at column cperm[k]
    (None: columns stay); rperm / cperm are int32 CUDA tensors."""
    _dev_check(rowptr, colidx, vals, rperm, cperm)
    assert rperm.dtype == torch.int32 and rperm.numel() == m
    assert cperm is None or (cperm.dtype == torch.int32 and cperm.numel() == n)
    nnz, code, dev = colidx.numel(), _DTYPE_CODE[vals.dtype], rowptr.device
    sz = ctypes.c_size_t(0)
    _check(_lib.spsyrk_permute(m, n, nnz, code, None, None, None, None, None, None, None, None, None, ctypes.byref(sz), None),
           "spsyrk_permute(size query)")
    ws = workspace if workspace is not None else _workspace(sz.value, dev)
    assert ws.numel() >= sz.value
    sz = ctypes.c_size_t(ws.numel())
    b_rowptr = torch.empty(m + 1, dtype=torch.int64, device=dev)
    b_colidx = torch.empty(max(nnz, 1), dtype=torch.int32, device=dev)
    b_vals = torch.empty(max(nnz, 1), dtype=vals.dtype, device=dev)
    _check(_lib.spsyrk_permute(m, n, nnz, code, _p(rowptr), _p(colidx), _p(vals), _p(rperm), _p(cperm), _p(b_rowptr),
                               _p(b_colidx), _p(b_vals), _p(ws), ctypes.byref(sz), _stream(stream)), "spsyrk_permute")
    return b_rowptr, b_colidx[:nnz], b_vals[:nnz]


def spsyrk_plan_partition(plan, parts, stream=None):
    """Row bounds (list of parts + 1 absolute row ids) of contiguous ranges of the plan's rows with
    near-equal work; worker p takes [bounds[p], bounds[p + 1])."""
    out = (ctypes.c_int64 * (parts + 1))()
    _check(_lib.spsyrk_plan_partition(plan._h, parts, out, _stream(stream)), "spsyrk_plan_partition")
    return list(out)


def spsyrk_symv(m, l_rowptr, l_colidx, l_vals, x, y=None, stream=None):
    """y = C x = C_L x + C_L^T x - D x from the lower triangle only (float64 or float32)."""
    _dev_check(l_rowptr, l_colidx, l_vals, x, y)
    assert x.dtype == l_vals.dtype and x.numel() == m
    if y is None:
        y = torch.empty(m, dtype=x.dtype, device=x.device)
    _check(_lib.spsyrk_symv(m, l_colidx.numel(), _DTYPE_CODE[l_vals.dtype], _p(l_rowptr), _p(l_colidx), _p(l_vals),
                            _p(x), _p(y), _stream(stream)), "spsyrk_symv")
    return y


def spsyrk_symm(m, l_rowptr, l_colidx, l_vals, x, y=None, stream=None):
    """Y = C X = C_L X + (X^T C_L)^T - D X for a dense row-major X of shape (m, p), from the lower triangle only."""
    _dev_check(l_rowptr, l_colidx, l_vals, x, y)
    assert x.dtype == l_vals.dtype and x.dim() == 2 and x.shape[0] == m
    p = x.shape[1]
    if y is None:
        y = torch.empty((m, p), dtype=x.dtype, device=x.device)
    _check(_lib.spsyrk_symm(m, p, l_colidx.numel(), _DTYPE_CODE[l_vals.dtype], _p(l_rowptr), _p(l_colidx), _p(l_vals),
                            _p(x), _p(y), _stream(stream)), "spsyrk_symm")
    return y


NOALLOC_MAX_ROWS = 1048576


def spsyrk_mirror_rowptr_noalloc(m, l_rowptr, l_colidx, f_rowptr, stream=None) -> int:
    """Row pointers of F = C_L + C_L^T - D into the caller's `f_rowptr` (m + 1 int64, CUDA) without
    any device allocation and without a workspace: the library's built-in scratch array is used,
    which caps m at NOALLOC_MAX_ROWS.  Returns nnz(F).  Calls that overlap on the GPU race on that
    array; the first call on a device should precede any stream capture."""
    _dev_check(l_rowptr, l_colidx, f_rowptr)
    assert f_rowptr.dtype == torch.int64 and f_rowptr.numel() >= m + 1
    nnz = ctypes.c_int64(0)
    _check(_lib.spsyrk_mirror_rowptr_noalloc(m, _p(l_rowptr), _p(l_colidx), _p(f_rowptr), ctypes.byref(nnz),
                                             _stream(stream)), "spsyrk_mirror_rowptr_noalloc")
    return nnz.value


def spsyrk_jaccard(m, row_begin, rows, a_rowptr, c_rowptr, c_colidx, c_counts, out=None, stream=None):
    _dev_check(a_rowptr, c_rowptr, c_colidx, c_counts, out)
    assert c_counts.dtype == torch.int32
    if out is None:
        out = torch.empty(c_counts.numel(), dtype=torch.float32, device=c_counts.device)
    _check(_lib.spsyrk_jaccard(m, row_begin, rows, _p(a_rowptr), _p(c_rowptr), _p(c_colidx), _p(c_counts), _p(out),
                               _stream(stream)), "spsyrk_jaccard")
    return out


def spsyrk_host_tril(m, n, rowptr, colidx, vals, mode=TRIL, pinned=True, out=None):
    """Whole path on HOST tensors through the host-buffer entry point.  Returns host tensors
    (c_rowptr, c_colidx, c_vals); the result buffers are pinned when `pinned`, or taken from
    `out` = (c_rowptr, c_colidx, c_vals) when given (they must be large enough)."""
    assert not rowptr.is_cuda and not colidx.is_cuda and not vals.is_cuda
    code = _DTYPE_CODE[vals.dtype]
    nnz = colidx.numel()
    sess = _vp()
    c_rowptr = out[0] if out is not None else torch.empty(m + 1, dtype=torch.int64, pin_memory=pinned)
    nnz_c = ctypes.c_int64(0)
    _check(_lib.spsyrk_host_tril(ctypes.byref(sess), m, n, nnz, _p(rowptr), _p(colidx), _p(vals), code, mode,
                                 _p(c_rowptr), ctypes.byref(nnz_c), None, None), "spsyrk_host_tril(symbolic)")
    if out is not None:
        c_colidx, c_vals = out[1], out[2]
        assert c_colidx.numel() >= nnz_c.value and c_vals.numel() >= nnz_c.value
    else:
        c_colidx = torch.empty(max(nnz_c.value, 1), dtype=torch.int32, pin_memory=pinned)
        c_vals = torch.empty(max(nnz_c.value, 1), dtype=vals.dtype, pin_memory=pinned)
    _check(_lib.spsyrk_host_tril(ctypes.byref(sess), m, n, nnz, None, None, None, code, mode, None, None,
                                 _p(c_colidx), _p(c_vals)), "spsyrk_host_tril(numeric)")
    return c_rowptr, c_colidx[:nnz_c.value], c_vals[:nnz_c.value]


def spsyrk_host_release_cache():
    """Free the device blocks spsyrk_host_tril keeps between calls on the current device."""
    _check(_lib.spsyrk_host_release_cache(), "spsyrk_host_release_cache")


# ------------------------------------------------------------------------------------------
# Convenience: the calls a user makes for one product, outputs allocated with torch.
# ------------------------------------------------------------------------------------------
def tril_syrk(m, n, rowptr, colidx, vals, mode=TRIL, row_begin=0, row_end=None, plan: Plan | None = None, stream=None,
              item_map=True):
    """plan -> (item map) -> symbolic -> numeric.  Returns (c_rowptr, c_colidx, c_vals, plan)."""
    if plan is None:
        plan = spsyrk_plan(m, n, rowptr, colidx, vals, mode, row_begin, row_end, stream)
    if item_map:
        spsyrk_plan_lend_map(plan, _workspace(spsyrk_plan_map_bytes(plan), rowptr.device))
    else:
        spsyrk_plan_lend_map(plan, None)
    c_rowptr = torch.empty(plan.rows + 1, dtype=torch.int64, device=rowptr.device)
    nnz = spsyrk_symbolic(plan, c_rowptr, stream)
    c_colidx = torch.empty(max(nnz, 1), dtype=torch.int32, device=rowptr.device)
    c_vals = torch.empty(max(nnz, 1), dtype=vals.dtype, device=rowptr.device)
    spsyrk_numeric(plan, c_rowptr, c_colidx, c_vals, stream)
    return c_rowptr, c_colidx[:nnz], c_vals[:nnz], plan
