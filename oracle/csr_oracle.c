/*
 * CPU oracle for CSR SpMV and CSR SpMM.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the GPU library is checked against.  Only the
 * test-suite, the smoke check and the benchmark's CPU-baseline leg may load it; the GPU library never
 * does, and nothing here is shared with it (own BF16 widening, own loops, plain C built by gcc).
 *
 * What it computes (paper, Appendix C, Table 6, task 12 "SpMV CSR" and task 13 "SpMM CSR": a matrix
 * A of shape (rows, cols) held as values[nnz], col_indices[nnz] and row_offsets[rows+1], the start of
 * each row in values; y = A x and C = A B with B of shape (cols, K), C of shape (rows, K)):
 *
 *   SpMV   y_ref[i]     = alpha * sum_{p in row i} vals[p] * x[col_idx[p]]        + beta * y0[i]
 *   SpMM   Y_ref[i,c]   = alpha * sum_{p in row i} vals[p] * B[col_idx[p], c]     + beta * Y0[i,c]
 *
 * The paper states the plain products; the alpha/beta form is this project's generalisation
 * (BLAS rule: beta == 0 means y0 is not read).  Every product and sum is done in double, one row
 * after the other, entries in storage order.  Beside each result the oracle returns
 * S_ref = sum_p |vals[p] * operand| (double), the scale the acceptance bound is stated against.
 * Inputs are the stored values: FP32, or BF16 bit patterns widened exactly.  Outputs stay double.
 *
 * nthreads > 1 only distributes whole rows over OpenMP threads (each row is still summed
 * sequentially by one thread), so results are bit-identical for any thread count.
 *
 * Parity pins (tests/test_oracle_pins.py): exact rational brute force on small dense matrices,
 * identity / diagonal closed forms, row sums of the 5- and 27-point stencils, the discrete Laplacian
 * of a linear function, linearity, SpMM-vs-SpMV column identities, the BF16 widening against an
 * independent library conversion over all 65536 patterns, and scipy's float64 CSR product.
 */
#include <stdint.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

/* BF16 is the upper half of an IEEE-754 binary32: widening appends sixteen zero bits. */
static double widen_bf16(uint16_t bits) {
  uint32_t u = (uint32_t)bits << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

static double load(const void* a, int64_t i, int dtype) {
  if (dtype == ORACLE_BF16) return widen_bf16(((const uint16_t*)a)[i]);
  return (double)((const float*)a)[i];
}

/* Exposed so that the widening itself can be pinned over every bit pattern. */
double oracle_bf16_to_double(uint16_t bits) { return widen_bf16(bits); }

int oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* y0 may be NULL when beta == 0.  Returns 0, or -1 on an unknown dtype. */
int oracle_spmv_csr(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx,
                    const void* vals, const void* x, const void* y0, double alpha, double beta, int dtype,
                    double* y_ref, double* S_ref, int nthreads) {
  (void)n; (void)nnz;
  if (dtype != ORACLE_F32 && dtype != ORACLE_BF16) return -1;
  int64_t i;
#pragma omp parallel for schedule(dynamic, 4096) num_threads(nthreads > 0 ? nthreads : 1)
  for (i = 0; i < m; ++i) {
    double acc = 0.0, S = 0.0;
    for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
      const double t = load(vals, p, dtype) * load(x, col_idx[p], dtype);
      acc += t;
      S += fabs(t);
    }
    y_ref[i] = alpha * acc + (beta == 0.0 ? 0.0 : beta * load(y0, i, dtype));
    if (S_ref) S_ref[i] = S;
  }
  return 0;
}

/* Rows listed in `rows` (nrows of them; NULL = all m rows in order).  Output row j of Y_ref / S_ref
 * (k entries each) belongs to matrix row rows[j].  B is (n, k) row-major, Y0 (m, k) row-major. */
int oracle_spmm_csr_rows(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr,
                         const int32_t* col_idx, const void* vals, const void* B, const void* Y0,
                         double alpha, double beta, int dtype, const int64_t* rows, int64_t nrows,
                         double* Y_ref, double* S_ref, int nthreads) {
  (void)n; (void)nnz;
  if (dtype != ORACLE_F32 && dtype != ORACLE_BF16) return -1;
  if (!rows) nrows = m;
  int64_t j;
#pragma omp parallel for schedule(dynamic, 64) num_threads(nthreads > 0 ? nthreads : 1)
  for (j = 0; j < nrows; ++j) {
    const int64_t i = rows ? rows[j] : j;
    for (int64_t c = 0; c < k; ++c) {
      double acc = 0.0, S = 0.0;
      for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
        const double t = load(vals, p, dtype) * load(B, (int64_t)col_idx[p] * k + c, dtype);
        acc += t;
        S += fabs(t);
      }
      Y_ref[j * k + c] = alpha * acc + (beta == 0.0 ? 0.0 : beta * load(Y0, i * k + c, dtype));
      if (S_ref) S_ref[j * k + c] = S;
    }
  }
  return 0;
}

int oracle_spmm_csr(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr,
                    const int32_t* col_idx, const void* vals, const void* B, const void* Y0, double alpha,
                    double beta, int dtype, double* Y_ref, double* S_ref, int nthreads) {
  return oracle_spmm_csr_rows(m, n, nnz, k, row_ptr, col_idx, vals, B, Y0, alpha, beta, dtype, 0, m, Y_ref,
                              S_ref, nthreads);
}

/* ------------------------------------------------------------------------------------------------
 * COO and ELL forms of the same products (paper, Appendix C, Table 6: tasks 8 / 9 "SpMV / SpMM COO" --
 * values[nnz], row_indices[nnz], col_indices[nnz] -- and tasks 14 / 15 "SpMV / SpMM ELL" -- values and
 * col_ids of size rows x max_nnz_per_row, padding positions marked with -1).  Readings: COO entries may
 * come in any order for the oracle (duplicates add; the sum is taken in storage order); ELL is row-major
 * (row i occupies [i*width, (i+1)*width)) and an entry is padding when its col_id is negative, whatever
 * its value holds.  k = 1 with B = x gives SpMV.
 * ---------------------------------------------------------------------------------------------- */
int oracle_spmm_coo(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_idx, const int32_t* col_idx,
                    const void* vals, const void* B, const void* Y0, double alpha, double beta, int dtype,
                    double* Y_ref, double* S_ref) {
  (void)n;
  if (dtype != ORACLE_F32 && dtype != ORACLE_BF16) return -1;
  for (int64_t i = 0; i < m * k; ++i) { Y_ref[i] = 0.0; if (S_ref) S_ref[i] = 0.0; }
  for (int64_t p = 0; p < nnz; ++p) {
    const int64_t i = row_idx[p];
    for (int64_t c = 0; c < k; ++c) {
      const double t = load(vals, p, dtype) * load(B, (int64_t)col_idx[p] * k + c, dtype);
      Y_ref[i * k + c] += t;
      if (S_ref) S_ref[i * k + c] += fabs(t);
    }
  }
  for (int64_t i = 0; i < m * k; ++i) Y_ref[i] = alpha * Y_ref[i] + (beta == 0.0 ? 0.0 : beta * load(Y0, i, dtype));
  return 0;
}

int oracle_spmm_ell(int64_t m, int64_t n, int64_t width, int64_t k, const int32_t* col_ids, const void* vals,
                    const void* B, const void* Y0, double alpha, double beta, int dtype, double* Y_ref, double* S_ref) {
  (void)n;
  if (dtype != ORACLE_F32 && dtype != ORACLE_BF16) return -1;
  for (int64_t i = 0; i < m; ++i)
    for (int64_t c = 0; c < k; ++c) {
      double acc = 0.0, S = 0.0;
      for (int64_t j = 0; j < width; ++j) {
        const int64_t p = i * width + j;
        if (col_ids[p] < 0) continue; /* padding */
        const double t = load(vals, p, dtype) * load(B, (int64_t)col_ids[p] * k + c, dtype);
        acc += t;
        S += fabs(t);
      }
      Y_ref[i * k + c] = alpha * acc + (beta == 0.0 ? 0.0 : beta * load(Y0, i * k + c, dtype));
      if (S_ref) S_ref[i * k + c] = S;
    }
  return 0;
}

/* CSC form (paper, Appendix C, Table 6: tasks 10 / 11 "SpMV / SpMM CSC" -- values[nnz], row_indices[nnz],
 * col_offsets[cols+1] = start of each column in values).  Column j contributes vals[p] * B[j, c] to row
 * row_idx[p]; the sum over a row is taken in column order, which is the storage order. */
int oracle_spmm_csc(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* col_ptr, const int32_t* row_idx,
                    const void* vals, const void* B, const void* Y0, double alpha, double beta, int dtype,
                    double* Y_ref, double* S_ref) {
  (void)nnz;
  if (dtype != ORACLE_F32 && dtype != ORACLE_BF16) return -1;
  for (int64_t i = 0; i < m * k; ++i) { Y_ref[i] = 0.0; if (S_ref) S_ref[i] = 0.0; }
  for (int64_t j = 0; j < n; ++j)
    for (int64_t p = col_ptr[j]; p < col_ptr[j + 1]; ++p) {
      const int64_t i = row_idx[p];
      for (int64_t c = 0; c < k; ++c) {
        const double t = load(vals, p, dtype) * load(B, j * k + c, dtype);
        Y_ref[i * k + c] += t;
        if (S_ref) S_ref[i * k + c] += fabs(t);
      }
    }
  for (int64_t i = 0; i < m * k; ++i) Y_ref[i] = alpha * Y_ref[i] + (beta == 0.0 ? 0.0 : beta * load(Y0, i, dtype));
  return 0;
}
