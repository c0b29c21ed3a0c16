"""Structure of the synthetic workloads: counts, ordering and distributions that the recipes fix."""
import numpy as np
import pytest

import gen


def check_csr(A):
    assert A.row_ptr.dtype == np.int32 and A.col_idx.dtype == np.int32 and A.vals.dtype == np.float32
    assert A.row_ptr[0] == 0 and A.row_ptr[-1] == A.nnz and A.row_ptr.shape[0] == A.m + 1
    assert np.all(np.diff(A.row_ptr) >= 0)
    assert A.col_idx.min() >= 0 and A.col_idx.max() < A.n


def sorted_unique_rows(A):
    d = np.diff(A.col_idx.astype(np.int64))
    row_start = np.zeros(A.nnz, bool)
    starts = A.row_ptr[:-1][np.diff(A.row_ptr) > 0]
    row_start[starts] = True
    return np.all((d > 0) | row_start[1:])


def test_lap2d_full_size():
    A = gen.lap2d(256)
    check_csr(A)
    assert A.m == 65536 and A.nnz == 326656
    assert sorted_unique_rows(A)
    L = np.diff(A.row_ptr)
    assert L.min() == 3 and L.max() == 5
    diag = A.vals[A.col_idx == np.repeat(np.arange(A.m), L)]
    assert np.all(diag == 4) and (A.vals == -1).sum() == A.nnz - A.m


def test_uniform_rows():
    A = gen.uniform_rows(1 << 14, 1 << 14, 16, 1002)
    check_csr(A)
    assert np.all(np.diff(A.row_ptr) == 16) and sorted_unique_rows(A)
    assert abs(A.vals.mean()) < 0.01 and abs(A.vals.std() - 1) < 0.01
    # columns uniform: mean near n/2, all 16 ranks present
    assert abs(A.col_idx.mean() / A.n - 0.5) < 0.01
    B = gen.uniform_rows(1 << 14, 1 << 14, 16, 1002)
    assert np.array_equal(A.col_idx, B.col_idx) and np.array_equal(A.vals, B.vals)   # seeded
    C = gen.uniform_rows(1 << 14, 1 << 14, 16, 7)
    assert not np.array_equal(A.col_idx, C.col_idx)
    # tiny n forces redraws; rows must still be duplicate-free
    D = gen.uniform_rows(500, 20, 16, 3)
    assert sorted_unique_rows(D)


def test_rmat_small_is_power_law():
    A = gen.rmat(16, 34_140_000 >> 6, 1003)
    check_csr(A)
    assert sorted_unique_rows(A)
    L = np.diff(A.row_ptr)
    assert L.argmax() == 0 and L.max() > 1000 and (L == 0).mean() > 0.3
    assert A.vals.min() > 0 and A.vals.max() <= 1
    assert 0.9 < A.nnz / (34_140_000 >> 6) <= 1.0


def test_rmat_relabel_keeps_degrees_and_moves_hubs():
    A = gen.rmat(14, 140_000, 7)
    B = gen.rmat(14, 140_000, 7, relabel=True)
    check_csr(B)
    assert sorted_unique_rows(B)
    assert A.nnz == B.nnz      # a bijection on vertex names merges no two distinct edges
    assert np.array_equal(np.sort(np.diff(A.row_ptr)), np.sort(np.diff(B.row_ptr)))
    assert np.array_equal(np.sort(np.bincount(A.col_idx, minlength=A.n)), np.sort(np.bincount(B.col_idx, minlength=B.n)))
    assert np.diff(B.row_ptr).argmax() != 0
    # hot columns are no longer packed at the low indices
    half = lambda M: (M.col_idx < M.n // 2).mean()
    assert half(A) > 0.7 and 0.35 < half(B) < 0.65


def test_stencil27():
    A = gen.stencil27(20, 1004)
    check_csr(A)
    assert A.nnz == 58 ** 3 and sorted_unique_rows(A)
    L = np.diff(A.row_ptr)
    assert set(np.unique(L)) == {8, 12, 18, 27}
    rows = np.repeat(np.arange(A.m), L)
    diag = A.col_idx == rows
    assert np.all(A.vals[diag] == 26)
    off = A.vals[~diag]
    assert abs(off.mean() + 1) < 1e-3 and abs(off.std() - 0.01) < 1e-3


def test_dense_samplers():
    u = gen.uniform(200000, -1.0, 1.0, 5, 0)
    assert u.min() >= -1 and u.max() < 1 and abs(u.mean()) < 0.01
    o = gen.uniform_open_low(200000, 5, 0)
    assert o.min() > 0 and o.max() <= 1
    z = gen.normal(200000, 5, 0)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01
    assert not np.array_equal(gen.uniform(100, -1, 1, 5, 0), gen.uniform(100, -1, 1, 5, 1))
    b = gen.to_bf16(z)
    assert np.max(np.abs(gen.bf16_to_f32(b) - z) / np.abs(z)) <= 2.0 ** -8


def test_algorithmic_bytes_formula():
    # the uniform 16-per-row workload at m = 2^20 in FP32 with beta != 0
    assert gen.algorithmic_bytes(1 << 20, 1 << 20, 1 << 24, 4, 0.5) == 150_994_948
    assert gen.algorithmic_bytes(1 << 20, 1 << 20, 1 << 24, 2, 0.5) == 111_149_060
    assert gen.algorithmic_bytes(65536, 65536, 326656, 4, 0.0) == 3_399_684


@pytest.mark.slow
def test_full_size_counts():
    assert gen.stencil27(160, 1004).nnz == 109_215_352
    A = gen.rmat(22, 34_140_000, 1003)
    L = np.diff(A.row_ptr)
    assert 33_400_000 < A.nnz < 33_700_000 and L.max() > 50_000 and L.argmax() == 0
