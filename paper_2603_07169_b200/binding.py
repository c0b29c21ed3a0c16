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
LIB_PATH = os.path.join(_HERE, "libb200sp.so")

F32, BF16 = 0, 1

EXPORTS = (
    "spmv_csr", "spmm_csr", "b200sp_plan_create", "b200sp_plan_destroy", "b200sp_plan_info", "b200sp_spmv",
    "b200sp_spmm", "spmv_csr_host", "spmm_csr_host", "b200sp_validate_csr", "b200sp_cache_clear",
    "b200sp_status_string", "b200sp_last_cuda_error", "b200sp_version", "b200sp_launch_count", "b200sp_set_option",
    "b200sp_check", "spmv_csr_noalloc", "b200sp_noalloc_max_items", "b200sp_probe_gather", "b200sp_spmv_naive", "b200sp_spmm_naive", "spmv_coo", "spmm_coo", "spmv_ell", "spmm_ell", "spmv_csc", "spmm_csc", "spmv_csr_vec_host",
)


class PlanInfo(ctypes.Structure):
    _fields_ = [("m", ctypes.c_int64), ("n", ctypes.c_int64), ("nnz", ctypes.c_int64),
                ("min_row_len", ctypes.c_int32), ("max_row_len", ctypes.c_int32),
                ("bin_rows", ctypes.c_int64 * 5), ("bin_nnz", ctypes.c_int64 * 5),
                ("spmv_kernel", ctypes.c_int32), ("spmv_tile_items", ctypes.c_int32), ("spmv_tiles", ctypes.c_int32),
                ("spmm_tile_nnz", ctypes.c_int32), ("spmm_tiles", ctypes.c_int32), ("scratch_bytes", ctypes.c_int64)]

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
        super().__init__("%s: %s (status %d)%s" % (where, msg, status, (": " + detail) if detail and status == 3 else ""))


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
        L.spmm_csr_host.argtypes = L.spmm_csr.argtypes
        L.b200sp_plan_create.argtypes = [ctypes.POINTER(p), i64, i64, i64, p, p]
        L.b200sp_plan_destroy.argtypes = [p]
        L.b200sp_plan_info.argtypes = [p, ctypes.POINTER(PlanInfo)]
        L.b200sp_spmv.argtypes = [p, p, p, p, p, f32, f32, i32, p]
        L.b200sp_spmm.argtypes = [p, i64, p, p, p, p, f32, f32, i32, p]
        L.b200sp_validate_csr.argtypes = [i64, i64, i64, p, p, p]
        L.b200sp_cache_clear.argtypes = []
        L.b200sp_cache_clear.restype = None
        L.b200sp_status_string.argtypes = [i32]
        L.b200sp_status_string.restype = ctypes.c_char_p
        L.b200sp_last_cuda_error.restype = ctypes.c_char_p
        L.b200sp_version.restype = i32
        L.b200sp_launch_count.restype = i64
        L.b200sp_set_option.argtypes = [ctypes.c_char_p, i32]
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


def spmv_csr(m, n, nnz, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    _ck(lib().spmv_csr(m, n, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _ptr(x), _ptr(y), alpha, beta, _dt(dtype),
                       _stream(stream)), "spmv_csr")


def spmm_csr(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    _ck(lib().spmm_csr(m, n, nnz, k, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _ptr(B), _ptr(Y), alpha, beta, _dt(dtype),
                       _stream(stream)), "spmm_csr")


def spmv_csr_noalloc(m, n, nnz, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    """SpMV for callers that may not allocate device memory: scratch comes from a fixed array inside the
    library (m + nnz <= b200sp_noalloc_max_items()); overlapping calls race on that array."""
    _ck(lib().spmv_csr_noalloc(m, n, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _ptr(x), _ptr(y), alpha, beta, _dt(dtype),
                               _stream(stream)), "spmv_csr_noalloc")


def spmv_coo(m, n, nnz, row_idx, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    _ck(lib().spmv_coo(m, n, nnz, _ptr(row_idx), _ptr(col_idx), _ptr(vals), _ptr(x), _ptr(y), alpha, beta, _dt(dtype), _stream(stream)), "spmv_coo")


def spmm_coo(m, n, nnz, k, row_idx, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    _ck(lib().spmm_coo(m, n, nnz, k, _ptr(row_idx), _ptr(col_idx), _ptr(vals), _ptr(B), _ptr(Y), alpha, beta, _dt(dtype), _stream(stream)), "spmm_coo")


def spmv_csc(m, n, nnz, col_ptr, row_idx, vals, x, y, alpha, beta, dtype, stream=None):
    _ck(lib().spmv_csc(m, n, nnz, _ptr(col_ptr), _ptr(row_idx), _ptr(vals), _ptr(x), _ptr(y), alpha, beta, _dt(dtype), _stream(stream)), "spmv_csc")


def spmm_csc(m, n, nnz, k, col_ptr, row_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    _ck(lib().spmm_csc(m, n, nnz, k, _ptr(col_ptr), _ptr(row_idx), _ptr(vals), _ptr(B), _ptr(Y), alpha, beta, _dt(dtype), _stream(stream)), "spmm_csc")


def spmv_ell(m, n, width, col_ids, vals, x, y, alpha, beta, dtype, stream=None):
    _ck(lib().spmv_ell(m, n, width, _ptr(col_ids), _ptr(vals), _ptr(x), _ptr(y), alpha, beta, _dt(dtype), _stream(stream)), "spmv_ell")


def spmm_ell(m, n, width, k, col_ids, vals, B, Y, alpha, beta, dtype, stream=None):
    _ck(lib().spmm_ell(m, n, width, k, _ptr(col_ids), _ptr(vals), _ptr(B), _ptr(Y), alpha, beta, _dt(dtype), _stream(stream)), "spmm_ell")


def b200sp_spmv_naive(m, n, nnz, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    _ck(lib().b200sp_spmv_naive(m, n, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _ptr(x), _ptr(y), alpha, beta, _dt(dtype),
                                _stream(stream)), "b200sp_spmv_naive")


def b200sp_spmm_naive(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    _ck(lib().b200sp_spmm_naive(m, n, nnz, k, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _ptr(B), _ptr(Y), alpha, beta, _dt(dtype),
                                _stream(stream)), "b200sp_spmm_naive")


def b200sp_probe_gather(table, table_elems, gathers, sink, stream=None):
    """Enqueues the random-gather probe (see include/b200sp.h); time it with CUDA events."""
    _ck(lib().b200sp_probe_gather(_ptr(table), table_elems, gathers, _ptr(sink), _stream(stream)), "b200sp_probe_gather")


def b200sp_noalloc_max_items() -> int:
    return lib().b200sp_noalloc_max_items()


def spmv_csr_host(m, n, nnz, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    _ck(lib().spmv_csr_host(m, n, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _ptr(x), _ptr(y), alpha, beta, _dt(dtype),
                            _stream(stream)), "spmv_csr_host")


def spmv_csr_vec_host(m, n, nnz, row_ptr, col_idx, vals, x_host, y_host, alpha, beta, dtype, stream=None):
    """Device-resident matrix, host x and y (one step of an iterative method)."""
    _ck(lib().spmv_csr_vec_host(m, n, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _ptr(x_host), _ptr(y_host), alpha, beta, _dt(dtype),
                                _stream(stream)), "spmv_csr_vec_host")


def spmm_csr_host(m, n, nnz, k, row_ptr, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    _ck(lib().spmm_csr_host(m, n, nnz, k, _ptr(row_ptr), _ptr(col_idx), _ptr(vals), _ptr(B), _ptr(Y), alpha, beta, _dt(dtype),
                            _stream(stream)), "spmm_csr_host")


def b200sp_plan_create(m, n, nnz, row_ptr, stream=None) -> int:
    out = ctypes.c_void_p()
    _ck(lib().b200sp_plan_create(ctypes.byref(out), m, n, nnz, _ptr(row_ptr), _stream(stream)), "b200sp_plan_create")
    return out.value


def b200sp_plan_destroy(plan):
    _ck(lib().b200sp_plan_destroy(plan), "b200sp_plan_destroy")


def b200sp_plan_info(plan) -> dict:
    info = PlanInfo()
    _ck(lib().b200sp_plan_info(plan, ctypes.byref(info)), "b200sp_plan_info")
    return info.as_dict()


def b200sp_spmv(plan, col_idx, vals, x, y, alpha, beta, dtype, stream=None):
    _ck(lib().b200sp_spmv(plan, _ptr(col_idx), _ptr(vals), _ptr(x), _ptr(y), alpha, beta, _dt(dtype), _stream(stream)), "b200sp_spmv")


def b200sp_spmm(plan, k, col_idx, vals, B, Y, alpha, beta, dtype, stream=None):
    _ck(lib().b200sp_spmm(plan, k, _ptr(col_idx), _ptr(vals), _ptr(B), _ptr(Y), alpha, beta, _dt(dtype), _stream(stream)), "b200sp_spmm")


def b200sp_validate_csr(m, n, nnz, row_ptr, col_idx, stream=None) -> int:
    """Returns the status (0 = consistent, 6 = inconsistent CSR) instead of raising on a bad matrix."""
    rc = lib().b200sp_validate_csr(m, n, nnz, _ptr(row_ptr), _ptr(col_idx), _stream(stream))
    if rc not in (0, 6):
        raise B200spError(rc, "b200sp_validate_csr")
    return rc


def b200sp_check(stream=None):
    """Synchronises the stream; raises B200spError(status 7) if a kernel gave up on a bounded wait."""
    _ck(lib().b200sp_check(_stream(stream)), "b200sp_check")


def b200sp_cache_clear():
    lib().b200sp_cache_clear()


def b200sp_version() -> int:
    return lib().b200sp_version()


def b200sp_launch_count() -> int:
    return lib().b200sp_launch_count()


def b200sp_set_option(name: str, value: int):
    _ck(lib().b200sp_set_option(name.encode(), value), "b200sp_set_option(%s)" % name)
