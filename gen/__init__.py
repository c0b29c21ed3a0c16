"""Seeded synthetic workloads for CSR SpMV / SpMM (host only).

This module serves both the CPU oracle's tests and the GPU path's tests and benchmark.  It holds
none of the SpMV / SpMM arithmetic: it only draws matrices and dense operands from a counter-based
generator and converts FP32 samples to BF16 storage.  The heavy generators are C++ (``gen.cpp``),
compiled on first use with g++; small adversarial matrices come from numpy's seeded generator.

The matrices are CSR as in the paper's benchmark task list (Appendix C, Table 6, tasks 12 and 13):
``vals`` (nnz), ``col_idx`` (nnz) and ``row_ptr`` (rows + 1, start of each row in ``vals``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.cpp")
_LIB = os.path.join(_HERE, "libb200sp_gen.so")


def build(force: bool = False) -> str:
    """Compile gen.cpp with g++ (OpenMP) if the shared object is missing or older than the source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, u64, i32, f32, f64, p = (ctypes.c_int64, ctypes.c_uint64, ctypes.c_int32, ctypes.c_float,
                                      ctypes.c_double, ctypes.c_void_p)
        lib.gen_uniform.argtypes = [i64, f32, f32, u64, u64, p]
        lib.gen_uniform_open_low.argtypes = [i64, u64, u64, p]
        lib.gen_normal.argtypes = [i64, f32, f32, u64, u64, p]
        lib.gen_f32_to_bf16.argtypes = [i64, p, p]
        lib.gen_lap2d_nnz.argtypes = [i64]
        lib.gen_lap2d_nnz.restype = i64
        lib.gen_lap2d.argtypes = [i64, p, p, p]
        lib.gen_uniform_rows.argtypes = [i64, i64, i32, u64, p, p, p]
        lib.gen_rmat.argtypes = [i32, i64, f64, f64, f64, u64, p, p, p]
        lib.gen_rmat.restype = i64
        lib.gen_rmat_relabel.argtypes = [i32, i64, f64, f64, f64, u64, p, p, p]
        lib.gen_rmat_relabel.restype = i64
        lib.gen_stencil27_nnz.argtypes = [i64]
        lib.gen_stencil27_nnz.restype = i64
        lib.gen_stencil27.argtypes = [i64, f32, f32, f32, u64, p, p, p]
        for name in ("gen_uniform", "gen_uniform_open_low", "gen_normal", "gen_f32_to_bf16", "gen_lap2d",
                     "gen_uniform_rows", "gen_stencil27"):
            getattr(lib, name).restype = None
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class CSR:
    """A CSR matrix with FP32 values (``vals``); ``vals_bf16()`` gives the BF16 storage patterns."""
    m: int
    n: int
    row_ptr: np.ndarray   # int32, m + 1
    col_idx: np.ndarray   # int32, nnz
    vals: np.ndarray      # float32, nnz
    name: str = ""

    @property
    def nnz(self) -> int:
        return int(self.col_idx.shape[0])

    def vals_bf16(self) -> np.ndarray:
        return to_bf16(self.vals)


# ------------------------------------------------------------------ dense operands
def uniform(n: int, lo: float, hi: float, seed: int, stream: int = 0) -> np.ndarray:
    """n FP32 samples lo + (hi - lo) * u, u a 24-bit fraction in [0, 1)."""
    out = np.empty(n, np.float32)
    _L().gen_uniform(n, lo, hi, seed, stream, _ptr(out))
    return out


def uniform_open_low(n: int, seed: int, stream: int = 0) -> np.ndarray:
    """n FP32 samples in (0, 1]: (u + 1) * 2^-24 with u a 24-bit integer."""
    out = np.empty(n, np.float32)
    _L().gen_uniform_open_low(n, seed, stream, _ptr(out))
    return out


def normal(n: int, seed: int, stream: int = 0, mean: float = 0.0, sigma: float = 1.0) -> np.ndarray:
    """n FP32 samples of N(mean, sigma^2) (Box-Muller in double, cast once)."""
    out = np.empty(n, np.float32)
    _L().gen_normal(n, mean, sigma, seed, stream, _ptr(out))
    return out


def to_bf16(a: np.ndarray) -> np.ndarray:
    """FP32 array -> uint16 array of BF16 bit patterns, round to nearest even (storage conversion)."""
    a = np.ascontiguousarray(a, np.float32)
    out = np.empty(a.shape, np.uint16)
    _L().gen_f32_to_bf16(a.size, _ptr(a), _ptr(out))
    return out


def bf16_to_f32(b: np.ndarray) -> np.ndarray:
    """uint16 BF16 patterns -> the FP32 values they denote (exact)."""
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


# ------------------------------------------------------------------ matrices
def lap2d(N: int) -> CSR:
    """2D 5-point Laplacian on an N x N grid: diagonal 4, existing neighbours -1, row index i*N + j."""
    nnz = _L().gen_lap2d_nnz(N)
    rp, ci, va = np.empty(N * N + 1, np.int32), np.empty(nnz, np.int32), np.empty(nnz, np.float32)
    _L().gen_lap2d(N, _ptr(rp), _ptr(ci), _ptr(va))
    return CSR(N * N, N * N, rp, ci, va, "lap2d_%d" % N)


def uniform_rows(m: int, n: int, per_row: int, seed: int) -> CSR:
    """Exactly per_row sorted distinct uniform columns in every row, values N(0, 1)."""
    assert per_row <= n
    nnz = m * per_row
    rp, ci, va = np.empty(m + 1, np.int32), np.empty(nnz, np.int32), np.empty(nnz, np.float32)
    _L().gen_uniform_rows(m, n, per_row, seed, _ptr(rp), _ptr(ci), _ptr(va))
    return CSR(m, n, rp, ci, va, "uniform%d_%d" % (per_row, m))


def rmat(scale: int, e_gen: int, seed: int, a: float = 0.57, b: float = 0.19, c: float = 0.19, relabel: bool = False) -> CSR:
    """R-MAT graph on 2^scale vertices from e_gen generated edges (sorted, duplicates dropped), values (0, 1].
    ``relabel`` renames every vertex by one pseudo-random bijection (same edges, same degrees, no index locality)."""
    m = 1 << scale
    rp, ci, va = np.empty(m + 1, np.int32), np.empty(e_gen, np.int32), np.empty(e_gen, np.float32)
    fn = _L().gen_rmat_relabel if relabel else _L().gen_rmat
    nnz = fn(scale, e_gen, a, b, c, seed, _ptr(rp), _ptr(ci), _ptr(va))
    return CSR(m, m, rp, ci[:nnz].copy(), va[:nnz].copy(), "rmat_%d%s" % (scale, "_relabel" if relabel else ""))


def stencil27(N: int, seed: int, diag: float = 26.0, off: float = -1.0, sigma: float = 0.01) -> CSR:
    """3D 27-point stencil on an N^3 grid, off-diagonals off + sigma*N(0,1) per entry, row (i*N + j)*N + l."""
    nnz = _L().gen_stencil27_nnz(N)
    m = N ** 3
    rp, ci, va = np.empty(m + 1, np.int32), np.empty(nnz, np.int32), np.empty(nnz, np.float32)
    _L().gen_stencil27(N, diag, off, sigma, seed, _ptr(rp), _ptr(ci), _ptr(va))
    return CSR(m, m, rp, ci, va, "stencil27_%d" % N)


def paper_uniform(rows: int, cols: int, density: float, seed: int) -> CSR:
    """The paper's sparse inputs (Table 6, tasks 12 / 13): nnz = floor(rows * cols * density) positions drawn
    uniformly without replacement over the whole matrix; values N(0, 1)."""
    nnz = int(rows * cols * density)
    rng = np.random.default_rng(seed)
    total = rows * cols
    pos = np.unique(rng.integers(0, total, int(nnz * 1.1) + 16))
    while pos.shape[0] < nnz:
        pos = np.unique(np.concatenate([pos, rng.integers(0, total, nnz)]))
    pos = np.sort(rng.permutation(pos)[:nnz])
    r, c = pos // cols, pos % cols
    rp = np.zeros(rows + 1, np.int64)
    np.add.at(rp, r + 1, 1)
    np.cumsum(rp, out=rp)
    va = rng.standard_normal(nnz).astype(np.float32)
    return CSR(rows, cols, rp.astype(np.int32), c.astype(np.int32), va, "paper_%dx%d" % (rows, cols))


def random_csr(m: int, n: int, row_lens, seed: int, sort_cols: bool = False, integer_vals: bool = False,
               allow_dup: bool = True) -> CSR:
    """Small adversarial matrix: given row lengths, columns uniform (duplicates allowed unless allow_dup
    is False), unsorted unless sort_cols; values N(0,1) or small integers in [-4, 4]."""
    rng = np.random.default_rng(seed)
    row_lens = np.asarray(row_lens, np.int64)
    assert row_lens.shape[0] == m
    rp = np.zeros(m + 1, np.int64)
    np.cumsum(row_lens, out=rp[1:])
    nnz = int(rp[-1])
    ci = np.empty(nnz, np.int32)
    for i in range(m):
        L = int(row_lens[i])
        if L == 0:
            continue
        if allow_dup:
            c = rng.integers(0, n, L)
        else:
            c = rng.choice(n, L, replace=False)
        if sort_cols:
            c = np.sort(c)
        ci[rp[i]:rp[i + 1]] = c
    if integer_vals:
        va = rng.integers(-4, 5, nnz).astype(np.float32)
    else:
        va = rng.standard_normal(nnz).astype(np.float32)
    return CSR(m, n, rp.astype(np.int32), ci, va, "random")


def csr_to_coo(A: CSR):
    """(row_idx, col_idx, vals) of a CSR matrix, entries in CSR order (sorted by row)."""
    rows = np.repeat(np.arange(A.m, dtype=np.int32), np.diff(A.row_ptr))
    return rows, A.col_idx.copy(), A.vals.copy()


def csr_to_csc(A: CSR):
    """(col_ptr, row_idx, vals) of the same matrix in CSC; entries of a column in ascending row order."""
    rows = np.repeat(np.arange(A.m, dtype=np.int64), np.diff(A.row_ptr))
    order = np.argsort(A.col_idx.astype(np.int64) * A.m + rows, kind="stable")
    cp = np.zeros(A.n + 1, np.int64)
    np.add.at(cp, A.col_idx.astype(np.int64) + 1, 1)
    np.cumsum(cp, out=cp)
    return cp.astype(np.int32), rows[order].astype(np.int32), A.vals[order].copy()


def csr_to_ell(A: CSR, width: Optional[int] = None, pad_value: float = -1.0):
    """(width, col_ids, vals), row-major m x width, padding marked with col_id = -1 (value -1 as in the paper's task text)."""
    L = np.diff(A.row_ptr)
    W = int(L.max()) if width is None else int(width)
    assert W >= (int(L.max()) if A.m else 0)
    col = np.full((A.m, W), -1, np.int32)
    val = np.full((A.m, W), pad_value, np.float32)
    j = np.arange(A.nnz, dtype=np.int64) - np.repeat(A.row_ptr[:-1].astype(np.int64), L)
    r = np.repeat(np.arange(A.m, dtype=np.int64), L)
    col[r, j] = A.col_idx
    val[r, j] = A.vals
    return W, col.ravel(), val.ravel()


# ------------------------------------------------------------------ the five measured workloads
@dataclass
class Workload:
    """One benchmark / parity configuration: matrix, dense operands (FP32 samples), scalars."""
    name: str
    A: CSR
    x: Optional[np.ndarray] = None     # SpMV operand (n)
    y0: Optional[np.ndarray] = None    # initial y (m) or Y (m*k) when beta != 0
    B: Optional[np.ndarray] = None     # SpMM operand (n*k row-major)
    k: int = 0
    alpha: float = 1.0
    beta: float = 0.0
    dtypes: tuple = ("f32",)
    note: str = ""


def workload(name: str, scale_down: int = 0) -> Workload:
    """The configurations measured by this project.  ``scale_down`` > 0 shrinks the problem (same
    structure and distributions, smaller m) for parity tests an oracle finishes in seconds.

    c1  2D 5-point Laplacian 256^2, x U[-1,1), alpha 1, beta 0                       (FP32)
    c2  m = n = 2^20, exactly 16 nnz/row, vals N(0,1), x and y0 U[-1,1), alpha 1.5, beta 0.5 (FP32, BF16)
    c3  R-MAT scale 22, 34.14 M generated edges, vals and x U(0,1], alpha 1, beta 0    (FP32)
    c3p the edges of c3 with every vertex renamed by one pseudo-random bijection (secondary measurement) (FP32)
    c3k64  the matrix of c3 times a dense B N(0,1) of n x 64: SpMM on uneven rows (secondary measurement) (FP32, BF16)
    c4  27-point stencil 160^3, diag 26, off -1 + N(0, 0.01^2), x N(0,1)               (BF16)
    c5k64 / c5k256  m = n = 2^19, 32 nnz/row, vals N(0,1), B N(0,1) n x k              (FP32, BF16)
    paper12_E / paper13_E  the paper's own SpMV / SpMM inputs: 2^E rows x 2048 columns at density 0.01 (K = 4096)
    """
    s = scale_down
    if name == "c1":
        N = 256 >> s
        A = lap2d(N)
        return Workload("c1", A, x=uniform(A.n, -1.0, 1.0, 1001, 10), dtypes=("f32",))
    if name == "c2":
        m = (1 << 20) >> (2 * s)
        A = uniform_rows(m, m, 16, 1002)
        return Workload("c2", A, x=uniform(m, -1.0, 1.0, 1002, 10), y0=uniform(m, -1.0, 1.0, 1002, 11),
                        alpha=1.5, beta=0.5, dtypes=("f32", "bf16"))
    if name == "c3":
        scale = 22 - 2 * s
        e_gen = 34_140_000 >> (2 * s)
        A = rmat(scale, e_gen, 1003)
        return Workload("c3", A, x=uniform_open_low(A.n, 1003, 10), dtypes=("f32",))
    if name == "c3p":
        scale = 22 - 2 * s
        e_gen = 34_140_000 >> (2 * s)
        A = rmat(scale, e_gen, 1003, relabel=True)
        return Workload("c3p", A, x=uniform_open_low(A.n, 1003, 10), dtypes=("f32",))
    if name == "c3k64":
        scale = 22 - 2 * s
        e_gen = 34_140_000 >> (2 * s)
        A = rmat(scale, e_gen, 1003)
        return Workload("c3k64", A, B=normal(A.n * 64, 1003, 12), k=64, dtypes=("f32", "bf16"))
    if name == "c4":
        N = 160 >> s
        A = stencil27(N, 1004)
        return Workload("c4", A, x=normal(A.n, 1004, 10), dtypes=("bf16",))
    if name in ("c5k64", "c5k256"):
        k = 64 if name == "c5k64" else 256
        m = (1 << 19) >> (2 * s)
        A = uniform_rows(m, m, 32, 1005)
        return Workload(name, A, B=normal(m * k, 1005, 10), k=k, dtypes=("f32", "bf16"))
    if name.startswith("paper12_") or name.startswith("paper13_"):
        # the paper's own inputs (Table 6, tasks 12 / 13): rows = 2^e, 2048 columns, density 0.01, K = 4096 for SpMM
        rows = 1 << int(name.split("_")[1])
        k = 4096 if name.startswith("paper13_") else 0
        A = paper_uniform(rows, 2048, 0.01, seed=rows + k)
        return Workload(name, A, x=uniform(2048, -1.0, 1.0, 7, 1), B=(normal(2048 * k, 7, 2) if k else None), k=k,
                        dtypes=("f32", "bf16"))
    raise ValueError("unknown workload %r" % name)


WORKLOADS = ("c1", "c2", "c3", "c4", "c5k64", "c5k256")


def algorithmic_bytes(m: int, n: int, nnz: int, e: int, beta: float, k: int = 0) -> int:
    """Bytes the operation must move when every CSR array and dense operand crosses HBM once:
    nnz*(4+e) + (m+1)*4 + n*e + m*e (+ m*e when beta != 0) for SpMV; dense terms times k for SpMM."""
    kk = max(k, 1)
    return nnz * (4 + e) + (m + 1) * 4 + n * kk * e + m * kk * e + (m * kk * e if beta != 0 else 0)
