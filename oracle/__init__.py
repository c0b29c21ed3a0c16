"""CPU oracle for CSR SpMV / SpMM -- TEST INFRASTRUCTURE ONLY.

A ctypes wrapper round ``csr_oracle.c`` (plain C, gcc, double accumulation).  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import this package; the GPU library never does and
shares no code with it.  See the header of ``csr_oracle.c`` for what is computed (paper, Appendix C,
Table 6, tasks 12 and 13, generalised with alpha / beta) and how it is pinned.

Acceptance bounds for a GPU result ``y`` against ``(y_ref, S_ref)``:
  FP32          |y - y_ref| <= 1e-5 * S_ref + 1e-30
  BF16 storage  |y - y_ref| <= 8e-3 * |y_ref| + 1e-5 * S_ref
``tolerance_ratio`` returns max(err / bound) and where it occurs; a pass is ratio <= 1.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csr_oracle.c")
_LIB = os.path.join(_HERE, "libcsr_oracle.so")

F32, BF16 = 0, 1
_DT = {"f32": F32, "bf16": BF16, F32: F32, BF16: BF16}


def build(force: bool = False) -> str:
    """Compile csr_oracle.c with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, f64, p = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        lib.oracle_spmv_csr.argtypes = [i64, i64, i64, p, p, p, p, p, f64, f64, i32, p, p, i32]
        lib.oracle_spmv_csr.restype = i32
        lib.oracle_spmm_csr_rows.argtypes = [i64, i64, i64, i64, p, p, p, p, p, f64, f64, i32, p, i64, p, p, i32]
        lib.oracle_spmm_csr_rows.restype = i32
        lib.oracle_spmm_coo.argtypes = [i64, i64, i64, i64, p, p, p, p, p, f64, f64, i32, p, p]
        lib.oracle_spmm_coo.restype = i32
        lib.oracle_spmm_csc.argtypes = [i64, i64, i64, i64, p, p, p, p, p, f64, f64, i32, p, p]
        lib.oracle_spmm_csc.restype = i32
        lib.oracle_spmm_ell.argtypes = [i64, i64, i64, i64, p, p, p, p, f64, f64, i32, p, p]
        lib.oracle_spmm_ell.restype = i32
        lib.oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
        lib.oracle_bf16_to_double.restype = f64
        lib.oracle_max_threads.restype = i32
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_L().oracle_max_threads())


def bf16_to_double(bits: int) -> float:
    return float(_L().oracle_bf16_to_double(bits))


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def _check(dtype, *arrays):
    want = np.float32 if _DT[dtype] == F32 else np.uint16
    for a in arrays:
        if a is not None and a.dtype != want:
            raise TypeError("dtype %r needs %s arrays (BF16 as uint16 bit patterns), got %s" % (dtype, want, a.dtype))


def spmv_csr(m, n, row_ptr, col_idx, vals, x, y0=None, alpha=1.0, beta=0.0, dtype="f32",
             nthreads: int = 1) -> Tuple[np.ndarray, np.ndarray]:
    """(y_ref, S_ref), both float64 of length m.  vals / x / y0 are float32, or uint16 BF16 patterns."""
    _check(dtype, vals, x, y0)
    row_ptr = np.ascontiguousarray(row_ptr, np.int32)
    col_idx = np.ascontiguousarray(col_idx, np.int32)
    assert row_ptr.shape[0] == m + 1 and x.shape[0] == n
    if beta != 0.0 and y0 is None:
        raise ValueError("beta != 0 needs y0")
    y, S = np.empty(m, np.float64), np.empty(m, np.float64)
    rc = _L().oracle_spmv_csr(m, n, col_idx.shape[0], _p(row_ptr), _p(col_idx), _p(vals), _p(x), _p(y0),
                              float(alpha), float(beta), _DT[dtype], _p(y), _p(S), nthreads)
    if rc != 0:
        raise RuntimeError("oracle_spmv_csr failed")
    return y, S


def spmm_csr(m, n, k, row_ptr, col_idx, vals, B, Y0=None, alpha=1.0, beta=0.0, dtype="f32", rows=None,
             nthreads: int = 1) -> Tuple[np.ndarray, np.ndarray]:
    """(Y_ref, S_ref), float64 of shape (len(rows) or m, k).  B is (n*k,) or (n, k) row-major."""
    _check(dtype, vals, B, Y0)
    row_ptr = np.ascontiguousarray(row_ptr, np.int32)
    col_idx = np.ascontiguousarray(col_idx, np.int32)
    assert B.size == n * k
    if beta != 0.0 and Y0 is None:
        raise ValueError("beta != 0 needs Y0")
    if rows is not None:
        rows = np.ascontiguousarray(rows, np.int64)
    nr = m if rows is None else rows.shape[0]
    Y, S = np.empty((nr, k), np.float64), np.empty((nr, k), np.float64)
    rc = _L().oracle_spmm_csr_rows(m, n, col_idx.shape[0], k, _p(row_ptr), _p(col_idx), _p(vals), _p(B), _p(Y0),
                                   float(alpha), float(beta), _DT[dtype], _p(rows), nr, _p(Y), _p(S), nthreads)
    if rc != 0:
        raise RuntimeError("oracle_spmm_csr failed")
    return Y, S


def spmm_coo(m, n, k, row_idx, col_idx, vals, B, Y0=None, alpha=1.0, beta=0.0, dtype="f32"):
    """COO form (entries in any order; duplicates add): (Y_ref, S_ref) of shape (m, k).  k = 1 with B = x is SpMV."""
    _check(dtype, vals, B, Y0)
    row_idx = np.ascontiguousarray(row_idx, np.int32)
    col_idx = np.ascontiguousarray(col_idx, np.int32)
    assert B.size == n * k and row_idx.shape == col_idx.shape
    if beta != 0.0 and Y0 is None:
        raise ValueError("beta != 0 needs Y0")
    Y, S = np.empty((m, k), np.float64), np.empty((m, k), np.float64)
    rc = _L().oracle_spmm_coo(m, n, col_idx.shape[0], k, _p(row_idx), _p(col_idx), _p(vals), _p(B), _p(Y0), float(alpha), float(beta),
                              _DT[dtype], _p(Y), _p(S))
    if rc != 0:
        raise RuntimeError("oracle_spmm_coo failed")
    return Y, S


def spmm_csc(m, n, k, col_ptr, row_idx, vals, B, Y0=None, alpha=1.0, beta=0.0, dtype="f32"):
    """CSC form (col_ptr of n + 1 entries, row_idx and vals in column-major order): (Y_ref, S_ref) of shape (m, k)."""
    _check(dtype, vals, B, Y0)
    col_ptr = np.ascontiguousarray(col_ptr, np.int32)
    row_idx = np.ascontiguousarray(row_idx, np.int32)
    assert col_ptr.shape[0] == n + 1 and B.size == n * k
    if beta != 0.0 and Y0 is None:
        raise ValueError("beta != 0 needs Y0")
    Y, S = np.empty((m, k), np.float64), np.empty((m, k), np.float64)
    rc = _L().oracle_spmm_csc(m, n, row_idx.shape[0], k, _p(col_ptr), _p(row_idx), _p(vals), _p(B), _p(Y0), float(alpha), float(beta),
                              _DT[dtype], _p(Y), _p(S))
    if rc != 0:
        raise RuntimeError("oracle_spmm_csc failed")
    return Y, S


def spmm_ell(m, n, width, k, col_ids, vals, B, Y0=None, alpha=1.0, beta=0.0, dtype="f32"):
    """ELL form (row-major m x width, padding where col_ids < 0): (Y_ref, S_ref) of shape (m, k)."""
    _check(dtype, vals, B, Y0)
    col_ids = np.ascontiguousarray(col_ids, np.int32)
    assert col_ids.size == m * width and vals.size == m * width and B.size == n * k
    if beta != 0.0 and Y0 is None:
        raise ValueError("beta != 0 needs Y0")
    Y, S = np.empty((m, k), np.float64), np.empty((m, k), np.float64)
    rc = _L().oracle_spmm_ell(m, n, width, k, _p(col_ids), _p(vals), _p(B), _p(Y0), float(alpha), float(beta), _DT[dtype], _p(Y), _p(S))
    if rc != 0:
        raise RuntimeError("oracle_spmm_ell failed")
    return Y, S


def tolerance_ratio(y, y_ref, S_ref, dtype="f32"):
    """max over entries of |y - y_ref| / bound, and the flat index where it occurs.  ``y`` is the GPU
    result as float32 (FP32 mode) or uint16 BF16 patterns (BF16 mode)."""
    if _DT[dtype] == BF16:
        yv = (np.ascontiguousarray(y, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        bound = 8e-3 * np.abs(y_ref) + 1e-5 * S_ref
    else:
        yv = np.asarray(y, np.float32).astype(np.float64)
        bound = 1e-5 * S_ref + 1e-30
    err = np.abs(yv.reshape(y_ref.shape) - y_ref)
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(err == 0.0, 0.0, err / bound)
    ratio = np.where(np.isnan(ratio), np.inf, ratio)
    if ratio.size == 0:
        return 0.0, -1
    i = int(np.argmax(ratio))
    return float(ratio.flat[i]), i
