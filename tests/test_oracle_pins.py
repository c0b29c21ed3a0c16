"""Pins for the CPU oracle: it is checked against things other than itself -- exact rational brute
force on dense matrices, closed forms, stencil identities, linearity, SpMM/SpMV identities, an
independent BF16 conversion, scipy's CSR product and a hand-worked fixture.  All run without a GPU."""
import os
from fractions import Fraction

import numpy as np
import pytest

import gen
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def frac(v):
    return Fraction(float(v))


def dense_exact(A, vals_f):
    """Densify a CSR matrix into exact rationals (duplicates add)."""
    D = [[Fraction(0)] * A.n for _ in range(A.m)]
    for i in range(A.m):
        for p in range(A.row_ptr[i], A.row_ptr[i + 1]):
            D[i][A.col_idx[p]] += frac(vals_f[p])
    return D


def stored(a, dtype):
    """(array handed to the oracle, exact float values it denotes)."""
    if dtype == "bf16":
        b = gen.to_bf16(a)
        return b, gen.bf16_to_f32(b)
    return a, a


# ---------------------------------------------------------------- brute force, exact rationals
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_spmv_vs_exact_dense_bruteforce(dtype, seed):
    rng = np.random.default_rng(seed)
    m, n = 13, 9
    lens = rng.integers(0, 7, m)
    lens[3] = 0
    A = gen.random_csr(m, n, lens, seed, sort_cols=False, allow_dup=True)
    x = rng.standard_normal(n).astype(np.float32)
    y0 = rng.standard_normal(m).astype(np.float32)
    v_s, v_f = stored(A.vals, dtype)
    x_s, x_f = stored(x, dtype)
    y_s, y_f = stored(y0, dtype)
    alpha, beta = 1.75, -0.5
    y, S = oracle.spmv_csr(m, n, A.row_ptr, A.col_idx, v_s, x_s, y_s, alpha, beta, dtype)
    # exact: walk the stored entries (not the dense matrix) so |.| sums are per stored entry
    for i in range(m):
        ex = Fraction(0)
        exS = Fraction(0)
        for p in range(A.row_ptr[i], A.row_ptr[i + 1]):
            t = frac(v_f[p]) * frac(x_f[A.col_idx[p]])
            ex += t
            exS += abs(t)
        ex = Fraction(alpha) * ex + Fraction(beta) * frac(y_f[i])
        tol = float(exS) * 2.0 ** -50 + abs(float(ex)) * 2.0 ** -51
        assert abs(Fraction(float(y[i])) - ex) <= Fraction(tol), (i, y[i], float(ex))
        assert abs(Fraction(float(S[i])) - exS) <= Fraction(float(exS) * 2.0 ** -50)
    # and against the densified matrix (duplicates merged): same product
    D = dense_exact(A, v_f)
    for i in range(m):
        ex = Fraction(alpha) * sum(D[i][j] * frac(x_f[j]) for j in range(n)) + Fraction(beta) * frac(y_f[i])
        assert abs(Fraction(float(y[i])) - ex) <= Fraction(float(S[i]) * 2.0 ** -49 + abs(float(ex)) * 2.0 ** -50)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_spmv_integer_data_is_exact(dtype):
    m, n = 40, 48
    rng = np.random.default_rng(7)
    A = gen.random_csr(m, n, rng.integers(0, 20, m), 11, integer_vals=True)
    x = rng.integers(-8, 9, n).astype(np.float32)
    y0 = rng.integers(-8, 9, m).astype(np.float32)
    v_s, _ = stored(A.vals, dtype)
    x_s, _ = stored(x, dtype)
    y_s, _ = stored(y0, dtype)
    y, S = oracle.spmv_csr(m, n, A.row_ptr, A.col_idx, v_s, x_s, y_s, 2.0, 0.5, dtype)
    D = np.zeros((m, n), np.int64)
    Dabs = np.zeros((m, n), np.int64)
    for i in range(m):
        for p in range(A.row_ptr[i], A.row_ptr[i + 1]):
            D[i, A.col_idx[p]] += int(A.vals[p])
    want = 2 * (D @ x.astype(np.int64)) + y0.astype(np.float64) / 2
    assert np.array_equal(y, want)
    wantS = np.array([sum(abs(int(A.vals[p]) * int(x[A.col_idx[p]])) for p in range(A.row_ptr[i], A.row_ptr[i + 1]))
                      for i in range(m)], np.float64)
    assert np.array_equal(S, wantS)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_spmm_vs_exact_dense_bruteforce(dtype):
    rng = np.random.default_rng(5)
    m, n, k = 11, 7, 5          # all different: a transposed B or Y index cannot pass
    A = gen.random_csr(m, n, rng.integers(0, 6, m), 21)
    B = rng.standard_normal(n * k).astype(np.float32)
    Y0 = rng.standard_normal(m * k).astype(np.float32)
    v_s, v_f = stored(A.vals, dtype)
    B_s, B_f = stored(B, dtype)
    Y_s, Y_f = stored(Y0, dtype)
    alpha, beta = -0.75, 2.0
    Y, S = oracle.spmm_csr(m, n, k, A.row_ptr, A.col_idx, v_s, B_s, Y_s, alpha, beta, dtype)
    D = dense_exact(A, v_f)
    for i in range(m):
        for c in range(k):
            ex = Fraction(alpha) * sum(D[i][j] * frac(B_f[j * k + c]) for j in range(n)) + Fraction(beta) * frac(Y_f[i * k + c])
            assert abs(Fraction(float(Y[i, c])) - ex) <= Fraction(float(S[i, c]) * 2.0 ** -49 + abs(float(ex)) * 2.0 ** -50)
    # S against a direct |.| sum
    for i in range(m):
        for c in range(k):
            exS = sum(abs(frac(v_f[p]) * frac(B_f[A.col_idx[p] * k + c])) for p in range(A.row_ptr[i], A.row_ptr[i + 1]))
            assert abs(Fraction(float(S[i, c])) - exS) <= Fraction(float(exS) * 2.0 ** -50)


# ---------------------------------------------------------------- closed forms
def test_identity_and_diagonal():
    n = 37
    rng = np.random.default_rng(0)
    x = rng.standard_normal(n).astype(np.float32)
    y0 = rng.standard_normal(n).astype(np.float32)
    d = rng.standard_normal(n).astype(np.float32)
    rp = np.arange(n + 1, dtype=np.int32)
    ci = np.arange(n, dtype=np.int32)
    alpha, beta = 0.5, 0.25
    y, S = oracle.spmv_csr(n, n, rp, ci, np.ones(n, np.float32), x, y0, alpha, beta)
    assert np.array_equal(y, alpha * x.astype(np.float64) + beta * y0.astype(np.float64))
    assert np.array_equal(S, np.abs(x.astype(np.float64)))
    y, S = oracle.spmv_csr(n, n, rp, ci, d, x, y0, alpha, beta)
    assert np.array_equal(y, alpha * (d.astype(np.float64) * x.astype(np.float64)) + beta * y0.astype(np.float64))
    # a permutation matrix moves entries (catches row/col mix-ups that a diagonal cannot)
    perm = rng.permutation(n).astype(np.int32)
    y, _ = oracle.spmv_csr(n, n, rp, perm, np.ones(n, np.float32), x)
    assert np.array_equal(y, x[perm].astype(np.float64))


def test_beta_zero_ignores_y0_and_empty_rows_are_zero():
    m, n = 6, 4
    A = gen.random_csr(m, n, [0, 2, 0, 3, 0, 0], 3)
    x = np.ones(n, np.float32)
    y_nan = np.full(m, np.nan, np.float32)
    y, S = oracle.spmv_csr(m, n, A.row_ptr, A.col_idx, A.vals, x, y_nan, 1.0, 0.0)
    assert np.all(np.isfinite(y))
    assert y[0] == 0.0 and y[2] == 0.0 and y[4] == 0.0 and S[0] == 0.0
    y, _ = oracle.spmv_csr(m, n, A.row_ptr, A.col_idx, A.vals, x, None, 1.0, 0.0)
    assert y[5] == 0.0


def test_row_sums_lap2d():
    N = 17
    A = gen.lap2d(N)
    assert A.nnz == 5 * N * N - 4 * N
    y, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, np.ones(A.n, np.float32))
    want = np.zeros((N, N))
    want[0, :] += 1; want[-1, :] += 1; want[:, 0] += 1; want[:, -1] += 1
    assert np.array_equal(y.reshape(N, N), want)          # 0 interior, 1 edges, 2 corners
    assert np.array_equal(S.reshape(N, N), 8 - want)


def test_row_sums_stencil27():
    N = 7
    A = gen.stencil27(N, seed=1, sigma=0.0)
    assert A.nnz == (3 * N - 2) ** 3
    y, _ = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, np.ones(A.n, np.float32))
    y = y.reshape(N, N, N)
    assert np.all(y[1:-1, 1:-1, 1:-1] == 0)               # 26 - 26
    assert y[0, 3, 3] == 9 and y[3, 0, 3] == 9 and y[3, 3, N - 1] == 9     # face: 26 - 17
    assert y[0, 0, 3] == 15 and y[0, 3, N - 1] == 15                       # edge: 26 - 11
    assert y[0, 0, 0] == 19 and y[N - 1, N - 1, N - 1] == 19               # corner: 26 - 7


def test_lap2d_of_linear_function():
    N = 12
    a, b, c = 3, -2, 5
    A = gen.lap2d(N)
    ii, jj = np.meshgrid(np.arange(N), np.arange(N), indexing="ij")
    u = (a * ii + b * jj + c).astype(np.float32).ravel()
    y, _ = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, u)
    y = y.reshape(N, N)
    assert np.all(y[1:-1, 1:-1] == 0)
    # boundary rows: the result equals the sum of u over the missing out-of-grid neighbours
    for j in range(1, N - 1):
        assert y[0, j] == a * (-1) + b * j + c
        assert y[N - 1, j] == a * N + b * j + c
    for i in range(1, N - 1):
        assert y[i, 0] == a * i + b * (-1) + c
        assert y[i, N - 1] == a * i + b * N + c
    assert y[0, 0] == (a * (-1) + c) + (b * (-1) + c)


def test_stencil27_of_linear_function():
    N = 6
    a, b, c, d = 2, -1, 3, 4
    A = gen.stencil27(N, seed=1, sigma=0.0)
    ii, jj, ll = np.meshgrid(np.arange(N), np.arange(N), np.arange(N), indexing="ij")
    u = (a * ii + b * jj + c * ll + d).astype(np.float32).ravel()
    y, _ = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, u)
    y = y.reshape(N, N, N)
    assert np.all(y[1:-1, 1:-1, 1:-1] == 0)
    # face i = 0: the nine missing neighbours at i = -1 sum to 9 * u(-1, j, l)
    assert y[0, 2, 3] == 9 * (a * (-1) + b * 2 + c * 3 + d)


# ---------------------------------------------------------------- linearity
def test_linearity_exact_on_integer_data():
    rng = np.random.default_rng(9)
    m, n = 50, 31
    A = gen.random_csr(m, n, rng.integers(0, 12, m), 4, integer_vals=True)
    x1 = rng.integers(-5, 6, n).astype(np.float32)
    x2 = rng.integers(-5, 6, n).astype(np.float32)
    y0 = rng.integers(-5, 6, m).astype(np.float32)
    f = lambda x, al=1.0, be=0.0: oracle.spmv_csr(m, n, A.row_ptr, A.col_idx, A.vals, x, y0, al, be)[0]
    assert np.array_equal(f(x1 + x2), f(x1) + f(x2))
    assert np.array_equal(f(4 * x1), 4 * f(x1))
    assert np.array_equal(f(x1, 2.0, 0.5), 2.0 * f(x1) + 0.5 * y0)
    assert np.array_equal(f(x1, 0.0, 3.0), 3.0 * y0.astype(np.float64))


# ---------------------------------------------------------------- SpMM identities
def test_spmm_columns_equal_spmv_and_selector():
    rng = np.random.default_rng(12)
    m, n, k = 23, 17, 6
    A = gen.random_csr(m, n, rng.integers(0, 9, m), 8)
    B = rng.standard_normal((n, k)).astype(np.float32)
    Y, S = oracle.spmm_csr(m, n, k, A.row_ptr, A.col_idx, A.vals, B.ravel())
    for c in range(k):
        y, s = oracle.spmv_csr(m, n, A.row_ptr, A.col_idx, A.vals, np.ascontiguousarray(B[:, c]))
        assert np.array_equal(Y[:, c], y) and np.array_equal(S[:, c], s)
    # k = 1 is SpMV
    Y1, _ = oracle.spmm_csr(m, n, 1, A.row_ptr, A.col_idx, A.vals, np.ascontiguousarray(B[:, 0]))
    assert np.array_equal(Y1[:, 0], Y[:, 0])
    # B = [I_k; 0] selects the first k columns of A (dense)
    E = np.zeros((n, k), np.float32)
    E[:k, :k] = np.eye(k, dtype=np.float32)
    Ye, _ = oracle.spmm_csr(m, n, k, A.row_ptr, A.col_idx, A.vals, E.ravel())
    D = np.zeros((m, n))
    for i in range(m):
        for p in range(A.row_ptr[i], A.row_ptr[i + 1]):
            D[i, A.col_idx[p]] += float(A.vals[p])
    assert np.allclose(Ye, D[:, :k], rtol=0, atol=1e-15)
    # sampled rows agree with the full product
    rows = np.array([22, 0, 7, 7], np.int64)
    Yr, Sr = oracle.spmm_csr(m, n, k, A.row_ptr, A.col_idx, A.vals, B.ravel(), rows=rows)
    assert np.array_equal(Yr, Y[rows]) and np.array_equal(Sr, S[rows])


# ---------------------------------------------------------------- BF16 widening, every pattern
def test_bf16_widening_all_patterns_vs_torch():
    import torch
    bits = np.arange(65536, dtype=np.int32)
    t = torch.from_numpy(bits.astype(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    for b in range(65536):
        v = oracle.bf16_to_double(b)
        if np.isnan(t[b]):
            assert np.isnan(v)
        else:
            assert v == t[b], b
    # and the generator's rounding against torch's round-to-nearest-even conversion
    x = gen.normal(100000, 3, 0)
    mine = gen.to_bf16(x)
    theirs = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(mine, theirs)


# ---------------------------------------------------------------- library routine at moderate size
@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_against_scipy_float64(name):
    import scipy.sparse as sp
    w = gen.workload(name, scale_down=2)
    A = w.A
    y0 = w.y0 if w.y0 is not None else None
    y, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, w.x, y0, w.alpha, w.beta, nthreads=4)
    M = sp.csr_matrix((A.vals.astype(np.float64), A.col_idx, A.row_ptr), shape=(A.m, A.n))
    want = w.alpha * (M @ w.x.astype(np.float64))
    if w.beta != 0:
        want = want + w.beta * y0.astype(np.float64)
    assert np.all(np.abs(want - y) <= 1e-13 * S + 1e-300)
    Mabs = sp.csr_matrix((np.abs(A.vals.astype(np.float64)), A.col_idx, A.row_ptr), shape=(A.m, A.n))
    assert np.all(np.abs(Mabs @ np.abs(w.x.astype(np.float64)) - S) <= 1e-13 * S)


def test_spmm_against_scipy_float64():
    import scipy.sparse as sp
    w = gen.workload("c5k64", scale_down=3)
    A = w.A
    Y, S = oracle.spmm_csr(A.m, A.n, w.k, A.row_ptr, A.col_idx, A.vals, w.B, nthreads=4)
    M = sp.csr_matrix((A.vals.astype(np.float64), A.col_idx, A.row_ptr), shape=(A.m, A.n))
    want = M @ w.B.astype(np.float64).reshape(A.n, w.k)
    assert np.all(np.abs(want - Y) <= 1e-13 * S + 1e-300)


def test_thread_count_does_not_change_bits():
    w = gen.workload("c3", scale_down=3)
    A = w.A
    y1, S1 = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, w.x, nthreads=1)
    y8, S8 = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, w.x, nthreads=8)
    assert np.array_equal(y1, y8) and np.array_equal(S1, S8)


# ---------------------------------------------------------------- hand-worked fixture
def _read_golden(path):
    d = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            d[key] = [float(v) for v in vals]
    return d


def test_hand_worked_fixture():
    g = _read_golden(os.path.join(GOLDEN, "spmv_hand_worked.txt"))
    m, n, k = int(g["m"][0]), int(g["n"][0]), int(g["k"][0])
    rp = np.array(g["row_ptr"], np.int32)
    ci = np.array(g["col_idx"], np.int32)
    va = np.array(g["vals"], np.float32)
    x = np.array(g["x"], np.float32)
    y0 = np.array(g["y0"], np.float32)
    for dtype in ("f32", "bf16"):
        cv = (lambda a: gen.to_bf16(a)) if dtype == "bf16" else (lambda a: a)
        y, S = oracle.spmv_csr(m, n, rp, ci, cv(va), cv(x), None, 1.0, 0.0, dtype)
        assert list(y) == g["Ax"] and list(S) == g["S"]
        y, _ = oracle.spmv_csr(m, n, rp, ci, cv(va), cv(x), cv(y0), g["alpha"][0], g["beta"][0], dtype)
        assert list(y) == g["y"]
        Y, _ = oracle.spmm_csr(m, n, k, rp, ci, cv(va), cv(np.array(g["B"], np.float32)), dtype=dtype)
        assert list(Y.ravel()) == g["AB"]


def test_tolerance_ratio_helper():
    y_ref = np.array([1.0, 0.0, -2.0])
    S = np.array([4.0, 0.0, 2.0])
    y = np.array([1.0 + 2e-5, 0.0, -2.0], np.float32)
    r, i = oracle.tolerance_ratio(y, y_ref, S, "f32")
    assert i == 0 and 0.4 < r < 0.6
    r, i = oracle.tolerance_ratio(np.array([1.0, 1e-20, -2.0], np.float32), y_ref, S, "f32")
    assert r > 1 and i == 1               # an empty row must be exactly zero
    yb = gen.to_bf16(np.array([1.0, 0.0, -2.0], np.float32))
    assert oracle.tolerance_ratio(yb, y_ref, S, "bf16")[0] == 0.0


# ---------------------------------------------------------------- COO and ELL forms
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_coo_and_ell_oracles_vs_exact_dense(dtype):
    rng = np.random.default_rng(31)
    m, n, k = 9, 6, 4
    A = gen.random_csr(m, n, [0, 3, 1, 0, 5, 2, 2, 0, 4], 5)
    B = rng.standard_normal(n * k).astype(np.float32)
    Y0 = rng.standard_normal(m * k).astype(np.float32)
    v_s, v_f = stored(A.vals, dtype)
    B_s, B_f = stored(B, dtype)
    Y_s, Y_f = stored(Y0, dtype)
    alpha, beta = 1.5, -0.25
    D = dense_exact(A, v_f)
    exact = [[Fraction(alpha) * sum(D[i][j] * frac(B_f[j * k + c]) for j in range(n)) + Fraction(beta) * frac(Y_f[i * k + c])
              for c in range(k)] for i in range(m)]
    # COO, entries shuffled (any order is legal for the definition)
    r, c, _ = gen.csr_to_coo(A)
    perm = rng.permutation(A.nnz)
    Yc, Sc = oracle.spmm_coo(m, n, k, r[perm], c[perm], np.ascontiguousarray(v_s[perm]), B_s, Y_s, alpha, beta, dtype)
    # ELL with extra padding columns; padded values are garbage on purpose
    W, ci, va = gen.csr_to_ell(A, width=7, pad_value=123.0)
    va_s, _ = stored(va, dtype)
    Ye, Se = oracle.spmm_ell(m, n, W, k, ci, va_s, B_s, Y_s, alpha, beta, dtype)
    Yr, Sr = oracle.spmm_csr(m, n, k, A.row_ptr, A.col_idx, v_s, B_s, Y_s, alpha, beta, dtype)
    for i in range(m):
        for cc in range(k):
            tol = Fraction(float(Sr[i, cc]) * 2.0 ** -48 + abs(float(exact[i][cc])) * 2.0 ** -50)
            assert abs(Fraction(float(Yc[i, cc])) - exact[i][cc]) <= tol
            assert abs(Fraction(float(Ye[i, cc])) - exact[i][cc]) <= tol
    assert np.array_equal(Ye, Yr) and np.array_equal(Se, Sr)          # ELL walks the entries in CSR order: bit-identical
    assert np.allclose(Sc, Sr, rtol=1e-14, atol=0)


def test_coo_ell_hand_worked_fixture():
    g = _read_golden(os.path.join(GOLDEN, "spmv_hand_worked.txt"))
    m, n = int(g["m"][0]), int(g["n"][0])
    rp = np.array(g["row_ptr"], np.int32)
    A = gen.CSR(m, n, rp, np.array(g["col_idx"], np.int32), np.array(g["vals"], np.float32))
    x = np.array(g["x"], np.float32)
    r, c, v = gen.csr_to_coo(A)
    y, S = oracle.spmm_coo(m, n, 1, r, c, v, x)
    assert list(y[:, 0]) == g["Ax"] and list(S[:, 0]) == g["S"]
    W, ci, va = gen.csr_to_ell(A)
    assert W == 4 and list(ci[:4]) == [0, 3, -1, -1] and list(ci[4:8]) == [-1] * 4
    y, S = oracle.spmm_ell(m, n, W, 1, ci, va, x)
    assert list(y[:, 0]) == g["Ax"] and list(S[:, 0]) == g["S"]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_csc_oracle_vs_exact_dense(dtype):
    rng = np.random.default_rng(41)
    m, n, k = 8, 11, 3                              # rows != cols != k: a swapped index cannot pass
    A = gen.random_csr(m, n, [2, 0, 5, 1, 3, 0, 4, 2], 6, allow_dup=False)
    cp, ri, va = gen.csr_to_csc(A)
    assert cp[-1] == A.nnz and np.all(np.diff(cp) >= 0)
    B = rng.standard_normal(n * k).astype(np.float32)
    Y0 = rng.standard_normal(m * k).astype(np.float32)
    v_s, v_f = stored(va, dtype)
    B_s, B_f = stored(B, dtype)
    Y_s, Y_f = stored(Y0, dtype)
    alpha, beta = -2.0, 0.5
    Y, S = oracle.spmm_csc(m, n, k, cp, ri, v_s, B_s, Y_s, alpha, beta, dtype)
    _, a_f = stored(A.vals, dtype)
    D = dense_exact(A, a_f)
    for i in range(m):
        for c in range(k):
            ex = Fraction(alpha) * sum(D[i][j] * frac(B_f[j * k + c]) for j in range(n)) + Fraction(beta) * frac(Y_f[i * k + c])
            assert abs(Fraction(float(Y[i, c])) - ex) <= Fraction(float(S[i, c]) * 2.0 ** -48 + abs(float(ex)) * 2.0 ** -50)
    # sorted unique columns: a row's entries come in the same order in both formats, so CSR and CSC agree bit for bit
    a_s, _ = stored(A.vals, dtype)
    Yr, Sr = oracle.spmm_csr(m, n, k, A.row_ptr, A.col_idx, a_s, B_s, Y_s, alpha, beta, dtype)
    As = gen.random_csr(m, n, [2, 0, 5, 1, 3, 0, 4, 2], 6, allow_dup=False, sort_cols=True)
    cp2, ri2, va2 = gen.csr_to_csc(As)
    a2_s, _ = stored(As.vals, dtype)
    v2_s, _ = stored(va2, dtype)
    Y1, S1 = oracle.spmm_csr(m, n, k, As.row_ptr, As.col_idx, a2_s, B_s, Y_s, alpha, beta, dtype)
    Y2, S2 = oracle.spmm_csc(m, n, k, cp2, ri2, v2_s, B_s, Y_s, alpha, beta, dtype)
    assert np.array_equal(Y1, Y2) and np.array_equal(S1, S2)
