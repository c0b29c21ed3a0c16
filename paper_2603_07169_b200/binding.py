"""Thin ctypes binding of libb200sp.so: argument marshalling only.

Every function here has the name and argument order of its C-ABI entry point (include/b200sp.h) and
passes raw pointers; all arithmetic runs in the CUDA kernels.  Tensors are torch CUDA tensors (used for
device memory and streams only) or, for the ``*_host`` calls, numpy / pinned torch CPU tensors.
The library is required: if libb200sp.so is missing or fails to load, importing raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
# B200SP_LIBRARY selects another build of the same library by file name (libb200sp_check.so: the checked build)
LIB_PATH = os.path.join(_HERE, os.environ.get("B200SP_LIBRARY", "libb200sp.so"))

F32, BF16 = 0, 1

EXPORTS = (
    "spmv_csr", "spmm_csr", "b200sp_plan_create", "b200sp_plan_destroy", "b200sp_plan_info", "b200sp_spmv",
    "b200sp_spmm", "spmv_csr_host", "spmm_csr_host", "b200sp_validate_csr", "b200sp_cache_clear",
    "b200sp_status_string", "b200sp_last_cuda_error", "b200sp_version", "b200sp_checked_build", "b200sp_launch_count", "b200sp_set_option", "b200sp_get_option",
    "b200sp_check", "b200sp_cache_drop", "spmv_csr_noalloc", "b200sp_noalloc_max_items", "b200sp_probe_gather", "b200sp_probe_gather_ex", "b200sp_probe_stream", "b200sp_probe_lines", "b200sp_probe_spmv_gather", "b200sp_spmv_naive", "b200sp_spmm_naive", "spmv_coo", "spmm_coo", "spmv_ell", "spmm_ell", "spmv_csc", "spmm_csc", "spmv_csr_vec_host",
)


class PlanInfo(ctypes.Structure):
    _fields_ = [("m", ctypes.c_int64), ("n", ctypes.c_int64), ("nnz", ctypes.c_int64),
                ("min_row_len", ctypes.c_int32), ("max_row_len", ctypes.c_int32),
                ("bin_rows", ctypes.c_int64 * 6), ("bin_nnz", ctypes.c_int64 * 6),
                ("spmv_kernel", ctypes.c_int32), ("spmv_tile_items", ctypes.c_int32), ("spmv_tiles", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("scratch_bytes", ctypes.c_int64)]

    def as_dict(self):
        d = {}
        for name, _ in self._fields_:
            v = getattr(self, name)
            d[name] = list(v) if hasattr(v, "__len__") else v
        return d


class B200spError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().b200sp_status_string(status).decode()
        detail = lib().b200sp_last_cuda_error().decode()
        super().__init__("%s: %s (status %d)%s" % (where, msg, status, (": " + detail) if detail and status in (3, 4) else ""))


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libb200sp.so is not built (%s); run `python -c 'import __graft_entry__ as g; g.build()'` "
                              "or `python -m paper_2603_07169_b200.build`" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        i64, i32, f32, p = ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_void_p
        L.spmv_csr.argtypes = [i64, i64, i64, p, p, p, p, p, f32, f32, i32, p]
        L.spmm_csr.argtypes = [i64, i64, i64, i64, p, p, p, p, p, f32, f32, i32, p]
        L.spmv_csr_host.argtypes = L.spmv_csr.argtypes
        L.spmv_csr_vec_host.argtypes = L.spmv_csr.argtypes
        L.spmv_csr_vec_host.restype = i32
        L.spmv_csr_noalloc.argtypes = L.spmv_csr.argtypes
        L.b200sp_spmv_naive.argtypes = L.spmv_csr.argtypes
        L.b200sp_spmv_naive.restype = i32
        L.b200sp_spmm_naive.argtypes = L.spmm_csr.argtypes
        L.b200sp_spmm_naive.restype = i32
        L.spmv_coo.argtypes = L.spmv_csr.argtypes
        L.spmm_coo.argtypes = L.spmm_csr.argtypes
        L.spmv_ell.argtypes = [i64, i64, i64, p, p, p, p, f32, f32, i32, p]
        L.spmm_ell.argtypes = [i64, i64, i64, i64, p, p, p, p, f32, f32, i32, p]
        L.spmv_csc.argtypes = L.spmv_csr.argtypes
        L.spmm_csc.argtypes = L.spmm_csr.argtypes
        for name in ("spmv_coo", "spmm_coo", "spmv_ell", "spmm_ell", "spmv_csc", "spmm_csc"):
            getattr(L, name).restype = i32
        L.spmv_csr_noalloc.restype = i32
        L.b200sp_noalloc_max_items.restype = i64
        L.b200sp_probe_gather.argtypes = [p, i64, i64, p, p]
        L.b200sp_probe_gather.restype = i32
        L.b200sp_probe_gather_ex.argtypes = [p, i64, i64, i32, i32, p, p]
        L.b200sp_probe_gather_ex.restype = i32
        L.b200sp_probe_stream.argtypes = [p, i64, p, p]
        L.b200sp_probe_stream.restype = i32
        L.b200sp_probe_lines.argtypes = [p, i64, i64, i32, i32, i32, p, p]
        L.b200sp_probe_lines.restype = i32
        L.b200sp_probe_spmv_gather.argtypes = [i64, p, p, p, i32, i32, p, p]
        L.b200sp_probe_spmv_gather.restype = i32
        L.spmm_csr_host.argtypes = L.spmm_csr.argtypes
        L.b200sp_plan_create.argtypes = [ctypes.POINTER(p), i64, i64, i64, p, p]
        L.b200sp_plan_destroy.argtypes = [p]
        L.b200sp_plan_info.argtypes = [p, ctypes.POINTER(PlanInfo)]
        L.b200sp_spmv.argtypes = [p, p, p, p, p, f32, f32, i32, p]
        L.b200sp_spmm.argtypes = [p, i64, p, p, p, p, f32, f32, i32, p]
        L.b200sp_validate_csr.argtypes = [i64, i64, i64, p, p, p]
        L.b200sp_cache_drop.argtypes = [p]
        L.b200sp_cache_drop.restype = i32
        L.b200sp_cache_clear.argtypes = []
        L.b200sp_cache_clear.restype = None
        L.b200sp_status_string.argtypes = [i32]
        L.b200sp_status_string.restype = ctypes.c_char_p
        L.b200sp_last_cuda_error.restype = ctypes.c_char_p
        L.b200sp_version.restype = i32
        L.b200sp_checked_build.restype = i32
        L.b200sp_launch_count.restype = i64
        L.b200sp_set_option.argtypes = [ctypes.c_char_p, i32]
        L.b200sp_get_option.argtypes = [ctypes.c_char_p, ctypes.POINTER(ctypes.c_int)]
        L.b200sp_get_option.restype = i32
        L.b200sp_check.argtypes = [p]
        L.b200sp_check.restype = i32
        for name in ("spmv_csr", "spmm_csr", "spmv_csr_host", "spmm_csr_host", "b200sp_plan_create", "b200sp_plan_destroy",
                     "b200sp_plan_info", "b200sp_spmv", "b200sp_spmm", "b200sp_validate_csr", "b200sp_set_option"):
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    """Raw address of a torch tensor or numpy array (None stays NULL)."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _esize(dtype) -> int:
    return 4 if _dt(dtype) == F32 else 2


def _dev(t, elems: int, esize: int, what: str, cur: Optional[int] = None) -> Optional[int]:
    """Address of a DEVICE operand.  The kernels dereference it on the GPU, and the library cannot tell a host address from
    a device address or see how long an array is, so this is the only place where a wrong tensor can be stopped: it must be
    a contiguous CUDA tensor on the current device with elements of `esize` bytes and at least `elems` of them.  Anything
    else raises B200spError(INVALID_ARG) before the library is entered.  None stays NULL (the library checks NULL
    against the sizes)."""
    if t is None:
        return None
    try:        # a few method calls only (this sits on the launch path of microsecond kernels); get_device() is -1 for a CPU tensor,
        #             and anything without these methods (a numpy array) is not a tensor
        ok = t.get_device() == (_current_device() if cur is None else cur) and t.element_size() == esize and t.numel() >= elems and t.is_contiguous()
    except AttributeError:
        ok = False
    if not ok:
        raise B200spError(1, "%s: expected a contiguous CUDA tensor on the current device with >= %d elements of %d bytes, got %s"
                          % (what, elems, esize, _describe(t)))
    return t.data_ptr()


_torch = None


def _current_device() -> int:
    """Index of the current CUDA device; -2 (which no tensor's device matches) on a machine without one."""
    global _torch
    if _torch is None:
        import torch
        _torch = torch
    try:
        return _torch.cuda.current_device()
    except (RuntimeError, AssertionError):
        return -2


def _host(t, elems: int, esize: int, what: str) -> Optional[int]:
    """Address of a HOST operand of the *_host entry points: a C-contiguous numpy array or a contiguous CPU tensor."""
    if t is None:
        return None
    if hasattr(t, "is_cuda"):
        ok = (not t.is_cuda) and t.is_contiguous() and t.element_size() == esize and (elems < 0 or t.numel() >= elems)
        addr = t.data_ptr() if ok else None
    else:
        ok = hasattr(t, "ctypes") and t.flags["C_CONTIGUOUS"] and t.itemsize == esize and (elems < 0 or t.size >= elems)
        addr = t.ctypes.data if ok else None
    if not ok:
        raise B200spError(1, "%s: expected a contiguous host array with >= %d elements of %d bytes, got %s"
                          % (what, elems, esize, _describe(t)))
    return addr


def _describe(t) -> str:
    try:
        if hasattr(t, "is_cuda"):
            return "torch tensor(device=%s, dtype=%s, numel=%d, contiguous=%s)" % (t.device, t.dtype, t.numel(), t.is_contiguous())
        return "%s(dtype=%s, size=%d)" % (type(t).__name__, getattr(t, "dtype", "?"), getattr(t, "size", -1))
    except Exception:  # pragma: no cover
        return repr(type(t))


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if hasattr(stream, "cuda_stream"):
        return stream.cuda_stream
    return int(stream)


def _dt(dtype) -> int:
    return {"f32": F32, "bf16": BF16, F32: F32, BF16: BF16}[dtype]


def _ck(status: int, where: str):
    if status != 0:
        raise B200spError(status, where)


def _csr_args(m, n, nnz, k, row_ptr, col_idx, vals, dense_in, dense_out, dtype, what, conv=_dev):
    e = _esize(dtype)
    kk = max(k, 1)
    if conv is _dev:
        cur = _current_device()          # once per call, not once per operand
        return (_dev(row_ptr, m + 1 if m > 0 else 0, 4, what, cur), _dev(col_idx, nnz, 4, what, cur), _dev(vals, nnz, e, what, cur),
                _dev(dense_in, n * kk if nnz > 0 else 0, e, what, cur), _dev(dense_out, m * kk, e, what, cur))
    return (conv(row_ptr, m + 1 if m > 0 else 0, 4, what + " row_ptr"), conv(col_idx, nnz, 4, what + " col_idx"), conv(vals, nnz, e, what + " vals"),
            conv(dense_in, n * kk if nnz > 0 else 0, e, what + " x/B"), conv(dense_out, m * kk, e, what + " y/Y"))


def spmv_csr(m, n, nnz, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    a = _csr_args(m, n, nnz, 0, row_ptr, col_idx, vals, x, y, dtype, "spmv_csr")
    _ck(lib().spmv_csr(m, n, nnz, a[0], a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "spmv_csr")


def spmm_csr(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    a = _csr_args(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, dtype, "spmm_csr")
    _ck(lib().spmm_csr(m, n, nnz, k, a[0], a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "spmm_csr")


def spmv_csr_noalloc(m, n, nnz, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    """SpMV for callers that may not allocate device memory: scratch comes from a fixed array inside the
    library (m + nnz <= b200sp_noalloc_max_items()); overlapping calls race on that array."""
    if 0 <= m + nnz <= b200sp_noalloc_max_items():
        a = _csr_args(m, n, nnz, 0, row_ptr, col_idx, vals, x, y, dtype, "spmv_csr_noalloc")
    else:   # refused by the library on the sizes alone: nothing is dereferenced
        a = [_ptr(t) for t in (row_ptr, col_idx, vals, x, y)]
    _ck(lib().spmv_csr_noalloc(m, n, nnz, a[0], a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "spmv_csr_noalloc")


def spmv_coo(m, n, nnz, row_idx, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    e = _esize(dtype)
    _ck(lib().spmv_coo(m, n, nnz, _dev(row_idx, nnz, 4, "spmv_coo row_idx"), _dev(col_idx, nnz, 4, "spmv_coo col_idx"),
                       _dev(vals, nnz, e, "spmv_coo vals"), _dev(x, n if nnz > 0 else 0, e, "spmv_coo x"), _dev(y, m, e, "spmv_coo y"),
                       alpha, beta, _dt(dtype), _stream(stream)), "spmv_coo")


def spmm_coo(m, n, nnz, k, row_idx, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    e = _esize(dtype)
    _ck(lib().spmm_coo(m, n, nnz, k, _dev(row_idx, nnz, 4, "spmm_coo row_idx"), _dev(col_idx, nnz, 4, "spmm_coo col_idx"),
                       _dev(vals, nnz, e, "spmm_coo vals"), _dev(B, n * k if nnz > 0 else 0, e, "spmm_coo B"), _dev(Y, m * k, e, "spmm_coo Y"),
                       alpha, beta, _dt(dtype), _stream(stream)), "spmm_coo")


def spmv_csc(m, n, nnz, col_ptr, row_idx, vals, x, y, alpha, beta, dtype, stream=None):
    e = _esize(dtype)
    _ck(lib().spmv_csc(m, n, nnz, _dev(col_ptr, n + 1, 4, "spmv_csc col_ptr"), _dev(row_idx, nnz, 4, "spmv_csc row_idx"),
                       _dev(vals, nnz, e, "spmv_csc vals"), _dev(x, n if nnz > 0 else 0, e, "spmv_csc x"), _dev(y, m, e, "spmv_csc y"),
                       alpha, beta, _dt(dtype), _stream(stream)), "spmv_csc")


def spmm_csc(m, n, nnz, k, col_ptr, row_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    e = _esize(dtype)
    _ck(lib().spmm_csc(m, n, nnz, k, _dev(col_ptr, n + 1, 4, "spmm_csc col_ptr"), _dev(row_idx, nnz, 4, "spmm_csc row_idx"),
                       _dev(vals, nnz, e, "spmm_csc vals"), _dev(B, n * k if nnz > 0 else 0, e, "spmm_csc B"), _dev(Y, m * k, e, "spmm_csc Y"),
                       alpha, beta, _dt(dtype), _stream(stream)), "spmm_csc")


def spmv_ell(m, n, width, col_ids, vals, x, y, alpha, beta, dtype, stream=None):
    e = _esize(dtype)
    _ck(lib().spmv_ell(m, n, width, _dev(col_ids, m * width, 4, "spmv_ell col_ids"), _dev(vals, m * width, e, "spmv_ell vals"),
                       _dev(x, n if m * width > 0 else 0, e, "spmv_ell x"), _dev(y, m, e, "spmv_ell y"), alpha, beta, _dt(dtype), _stream(stream)), "spmv_ell")


def spmm_ell(m, n, width, k, col_ids, vals, B, Y, alpha, beta, dtype, stream=None):
    e = _esize(dtype)
    _ck(lib().spmm_ell(m, n, width, k, _dev(col_ids, m * width, 4, "spmm_ell col_ids"), _dev(vals, m * width, e, "spmm_ell vals"),
                       _dev(B, n * k if m * width > 0 else 0, e, "spmm_ell B"), _dev(Y, m * k, e, "spmm_ell Y"), alpha, beta, _dt(dtype),
                       _stream(stream)), "spmm_ell")


def b200sp_spmv_naive(m, n, nnz, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    a = _csr_args(m, n, nnz, 0, row_ptr, col_idx, vals, x, y, dtype, "b200sp_spmv_naive")
    _ck(lib().b200sp_spmv_naive(m, n, nnz, a[0], a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "b200sp_spmv_naive")


def b200sp_spmm_naive(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    a = _csr_args(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, dtype, "b200sp_spmm_naive")
    _ck(lib().b200sp_spmm_naive(m, n, nnz, k, a[0], a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "b200sp_spmm_naive")


def b200sp_probe_gather(table, table_elems, gathers, sink, stream=None):
    """Enqueues the random-gather probe (see include/b200sp_tuning.h); time it with CUDA events."""
    _ck(lib().b200sp_probe_gather(_dev(table, table_elems, 4, "probe table"), table_elems, gathers, _dev(sink, 1, 4, "probe sink"),
                                  _stream(stream)), "b200sp_probe_gather")


def b200sp_probe_gather_ex(table, table_elems, gathers, elem_bytes, in_shared_memory, sink, stream=None):
    _ck(lib().b200sp_probe_gather_ex(_dev(table, table_elems, elem_bytes, "probe table"), table_elems, gathers, elem_bytes, in_shared_memory,
                                     _dev(sink, 1, 4, "probe sink"), _stream(stream)), "b200sp_probe_gather_ex")


def b200sp_probe_stream(buf, nbytes, sink, stream=None):
    _ck(lib().b200sp_probe_stream(_dev(buf, nbytes // max(buf.element_size(), 1), buf.element_size(), "probe buffer"), nbytes,
                                  _dev(sink, 1, 4, "probe sink"), _stream(stream)), "b200sp_probe_stream")


def b200sp_probe_lines(buf, lines, reads, sink, in_flight=4, to_shared_memory=0, stream=None, group_lanes=8):
    _ck(lib().b200sp_probe_lines(_dev(buf, lines * 128 // max(buf.element_size(), 1), buf.element_size(), "probe buffer"), lines, reads,
                                 in_flight, to_shared_memory, group_lanes, _dev(sink, 1, 4, "probe sink"), _stream(stream)), "b200sp_probe_lines")


def b200sp_probe_spmv_gather(nnz, col_idx, vals, x, dtype, unused_smem_kb, out, stream=None):
    code = _dt(dtype)
    esize = 4 if code == 0 else 2
    _ck(lib().b200sp_probe_spmv_gather(nnz, _dev(col_idx, nnz, 4, "col_idx"), _dev(vals, nnz, esize, "vals"), _dev(x, 1, esize, "x"), code,
                                       unused_smem_kb, _dev(out, 1, 4, "probe out"), _stream(stream)), "b200sp_probe_spmv_gather")


def b200sp_noalloc_max_items() -> int:
    return lib().b200sp_noalloc_max_items()


def spmv_csr_host(m, n, nnz, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    a = _csr_args(m, n, nnz, 0, row_ptr, col_idx, vals, x, y, dtype, "spmv_csr_host", conv=_host)
    _ck(lib().spmv_csr_host(m, n, nnz, a[0], a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "spmv_csr_host")


def spmv_csr_vec_host(m, n, nnz, row_ptr, col_idx, vals, x_host, y_host, alpha, beta, dtype, stream=None):
    """Device-resident matrix, host x and y (one step of an iterative method)."""
    e = _esize(dtype)
    _ck(lib().spmv_csr_vec_host(m, n, nnz, _dev(row_ptr, m + 1 if m > 0 else 0, 4, "spmv_csr_vec_host row_ptr"),
                                _dev(col_idx, nnz, 4, "spmv_csr_vec_host col_idx"), _dev(vals, nnz, e, "spmv_csr_vec_host vals"),
                                _host(x_host, n if nnz > 0 else 0, e, "spmv_csr_vec_host x"), _host(y_host, m, e, "spmv_csr_vec_host y"),
                                alpha, beta, _dt(dtype), _stream(stream)), "spmv_csr_vec_host")


def spmm_csr_host(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    a = _csr_args(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, dtype, "spmm_csr_host", conv=_host)
    _ck(lib().spmm_csr_host(m, n, nnz, k, a[0], a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "spmm_csr_host")


def b200sp_plan_create(m, n, nnz, row_ptr, stream=None) -> int:
    out = ctypes.c_void_p()
    _ck(lib().b200sp_plan_create(ctypes.byref(out), m, n, nnz, _dev(row_ptr, m + 1 if m > 0 else 0, 4, "b200sp_plan_create row_ptr"),
                                 _stream(stream)), "b200sp_plan_create")
    return out.value


def b200sp_plan_destroy(plan):
    _ck(lib().b200sp_plan_destroy(plan), "b200sp_plan_destroy")


def b200sp_plan_info(plan) -> dict:
    info = PlanInfo()
    _ck(lib().b200sp_plan_info(plan, ctypes.byref(info)), "b200sp_plan_info")
    return info.as_dict()


def b200sp_spmv(plan, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    I = b200sp_plan_info(plan)      # the plan knows m, n, nnz
    a = _csr_args(I["m"], I["n"], I["nnz"], 0, None, col_idx, vals, x, y, dtype, "b200sp_spmv")
    _ck(lib().b200sp_spmv(plan, a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "b200sp_spmv")


def b200sp_spmm(plan, k, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    I = b200sp_plan_info(plan)
    a = _csr_args(I["m"], I["n"], I["nnz"], k, None, col_idx, vals, B, Y, dtype, "b200sp_spmm")
    _ck(lib().b200sp_spmm(plan, k, a[1], a[2], a[3], a[4], alpha, beta, _dt(dtype), _stream(stream)), "b200sp_spmm")


def b200sp_validate_csr(m, n, nnz, row_ptr, col_idx, stream=None) -> int:
    """Returns the status (0 = consistent, 6 = inconsistent CSR) instead of raising on a bad matrix."""
    rc = lib().b200sp_validate_csr(m, n, nnz, _dev(row_ptr, m + 1, 4, "b200sp_validate_csr row_ptr"),
                                   _dev(col_idx, nnz, 4, "b200sp_validate_csr col_idx"), _stream(stream))
    if rc not in (0, 6):
        raise B200spError(rc, "b200sp_validate_csr")
    return rc


def b200sp_check(stream=None):
    """Synchronises the stream; raises B200spError(status 7) if a kernel gave up on a bounded wait."""
    _ck(lib().b200sp_check(_stream(stream)), "b200sp_check")


def b200sp_cache_clear():
    lib().b200sp_cache_clear()


def b200sp_cache_drop(key):
    """Forgets what the one-shot calls cached under this array's address (a row_ptr / row_idx / col_ptr tensor or array).
    Call it before freeing or rewriting such an array: the caches are keyed on addresses, and an allocator that hands
    the address out again would otherwise revive a stale plan."""
    _ck(lib().b200sp_cache_drop(_ptr(key)), "b200sp_cache_drop")


def b200sp_version() -> int:
    return lib().b200sp_version()


def b200sp_checked_build() -> int:
    return lib().b200sp_checked_build()


def b200sp_launch_count() -> int:
    return lib().b200sp_launch_count()


def b200sp_set_option(name: str, value: int):
    _ck(lib().b200sp_set_option(name.encode(), value), "b200sp_set_option(%s)" % name)


def b200sp_get_option(name: str) -> int:
    out = ctypes.c_int(0)
    _ck(lib().b200sp_get_option(name.encode(), ctypes.byref(out)), "b200sp_get_option(%s)" % name)
    return out.value
