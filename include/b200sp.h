/*
 * b200sp -- CSR sparse matrix-vector and sparse-times-dense products for NVIDIA B200 (sm_100a).
 *
 * C ABI of the shared library libb200sp.so.  Plain pointers and sizes only; no exception crosses
 * this boundary; every function returns a b200sp_status (0 = success) unless stated otherwise.
 *
 * Operations (paper: Appendix C, Table 6, task 12 "SpMV CSR" and task 13 "SpMM CSR", which define
 * A of shape (rows, cols) by values[nnz], col_indices[nnz] and row_offsets[rows + 1] = start of each
 * row in values, with y = A x and C = A B, B of shape (cols, K), C of shape (rows, K)).  This
 * library computes the BLAS-style generalisation
 *
 *     SpMV:  y = alpha * A * x + beta * y            x: n entries, y: m entries
 *     SpMM:  Y = alpha * A * B + beta * Y            B: n x k, Y: m x k, both row-major, leading dim k
 *
 * in FP32, or with BF16 storage and FP32 accumulation (B200SP_BF16: vals, x / B and y / Y hold raw
 * 16-bit bfloat16 patterns; alpha and beta stay FP32; every product and sum is FP32; one
 * round-to-nearest-even conversion at the final store).
 *
 * Conventions common to all entry points
 *  - Indices are 0-based int32; sizes are int64 with m, n, nnz < 2^31; row_ptr[0] = 0,
 *    row_ptr[m] = nnz, row_ptr non-decreasing, 0 <= col_idx[p] < n.  Content is NOT checked on the
 *    hot path (b200sp_validate_csr does it on request).  Columns may be unsorted; duplicates add.
 *  - Unless a function says "host", every array pointer is a DEVICE pointer on the current device,
 *    owned by the caller, which keeps it alive and unmodified until the stream work has finished.
 *    col_idx, vals, x / B and y / Y must be 16-byte aligned, row_ptr 4-byte aligned.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls enqueue
 *    work and return without synchronising, except where stated (plan creation reads back a few
 *    hundred bytes and synchronises the stream once).
 *  - beta == 0: y / Y is write-only (its old contents, NaN included, are ignored).  alpha == 0 or
 *    nnz == 0: y = beta * y without reading A.  m == 0: nothing is done.  x / B must not alias y / Y.
 *  - The compute kernels are launched with programmatic stream serialisation (option "pdl"): a kernel waits for the
 *    stream's earlier work (griddepcontrol.wait) before its first memory access, then lets the next kernel of the
 *    stream be scheduled behind it.  Ordinary launches that follow see ordinary stream order.  A caller that launches
 *    its own next kernel with the same attribute must call cudaGridDependencySynchronize() in it before reading y / Y.
 *  - Results are deterministic: the same inputs give bit-identical outputs on every call (no
 *    floating-point atomics; rows cut by a tile boundary are completed in a fixed order).
 *  - Errors: host-detectable problems (negative or too large sizes, NULL pointer with non-zero
 *    size, unknown dtype, k <= 0, misaligned pointer) return B200SP_ERR_INVALID_ARG and launch
 *    nothing; a device that is not compute capability 10.x returns B200SP_ERR_ARCH; a failing CUDA
 *    call returns B200SP_ERR_CUDA and its message is kept for b200sp_last_cuda_error().
 *  - Device memory the library needs (plan scratch, the staging buffers of the "host" entry
 *    points, and per-call scratch for SpMM, taken and returned in the order of `stream`: on matrices
 *    with very uneven rows a few bytes per 1024 nonzeros and dense column; on matrices with so few
 *    columns that a slice of B is kept in shared memory a re-laid copy of A, about (2 + bytes per
 *    value) * (nnz + 3 m) bytes, plus 8 m bytes kept with the plan) comes from a
 *    stream-ordered memory pool of its own, one per device, created at first use.  The pool keeps up to 1 GiB of freed memory for the next call (option "pool_keep_mb",
 *    read when the pool is created); b200sp_cache_clear hands all unused pool memory back.
 *  - There is no CPU fallback: without a B200 the compute entry points fail.
 */
#ifndef B200SP_H_
#define B200SP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { B200SP_F32 = 0, B200SP_BF16 = 1 } b200sp_dtype;

typedef enum {
  B200SP_OK = 0,
  B200SP_ERR_INVALID_ARG = 1,
  B200SP_ERR_UNSUPPORTED = 2,
  B200SP_ERR_CUDA = 3,
  B200SP_ERR_ALLOC = 4,
  B200SP_ERR_ARCH = 5,
  B200SP_ERR_BAD_CSR = 6,
  B200SP_ERR_TIMEOUT = 7,
  B200SP_ERR_TOO_LARGE = 8
} b200sp_status;

/* Opaque: row statistics, row bins, nnz-balanced tile splits and the scratch the kernels need. */
typedef struct b200sp_plan b200sp_plan;

/* Row-length bins of the plan pass: rows of length 0, 1-4, 5-32, 33-128, 129-1024 and > 1024. */
#define B200SP_NUM_BINS 6

/* What the plan pass found (b200sp_plan_info).  All counts are exact integers. */
typedef struct {
  int64_t m, n, nnz;
  int32_t min_row_len, max_row_len;
  int64_t bin_rows[B200SP_NUM_BINS];  /* rows per length bin */
  int64_t bin_nnz[B200SP_NUM_BINS];   /* nonzeros held by the rows of each bin */
  int32_t spmv_kernel;                /* 0 = merge-tile kernel (rows + nnz balanced), 1 = row-direct kernel,
                                         2 = uniform-row sub-warp kernel, 3 = sub-warp-per-row kernel (small problems) */
  int32_t spmv_tile_items;            /* merge items (rows + nonzeros) per merge tile */
  int32_t spmv_tiles;                 /* number of merge tiles */
  int32_t reserved;                   /* 0 */
  int64_t scratch_bytes;              /* device memory held by the plan */
} b200sp_plan_info_t;

/* ---- one-shot calls -------------------------------------------------------------------------
 * Task 12 / task 13 of the paper's Table 6 with alpha and beta.  The first call for a given
 * (device, row_ptr, m, n, nnz) builds a plan (see b200sp_plan_create; synchronises the stream once)
 * and caches it inside the library; later calls with the same key reuse it, so the CONTENTS of
 * row_ptr must not change while the plan is cached.  The key is the ADDRESS: if the caller frees row_ptr
 * and an allocator hands the same address out again for another matrix with the same m, n and nnz (a
 * caching allocator does this readily), the stale plan would be used and the result would be wrong
 * without any error.  Call b200sp_cache_drop(row_ptr) before releasing or rewriting a row_ptr array (or
 * b200sp_cache_clear for everything), or use the plan API, which has no hidden state.  The cache holds
 * at most 1024 plans and drops the least recently used one beyond that (dropping synchronises the device).
 * Two calls that use the same cached plan must not overlap on the GPU (they share its scratch).
 * dtype is a b200sp_dtype. */
int spmv_csr(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx,
             const void* vals, const void* x, void* y, float alpha, float beta, int dtype, void* stream);

int spmm_csr(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr, const int32_t* col_idx,
             const void* vals, const void* B, void* Y, float alpha, float beta, int dtype, void* stream);

/* ---- plan API --------------------------------------------------------------------------------
 * The plan pass depends on the sparsity pattern's row structure only (row_ptr): it computes the
 * row-length statistics and bins, chooses the kernels, and computes the nnz-balanced split points
 * (a merge-path search over rows + nonzeros) and the lists of rows of 129-1024 and of more than 1024 nonzeros that
 * SpMM treats separately, all on the device.  From the same statistics it decides whether SpMM gives every row to a
 * group of eight lanes (even rows) or cuts the nonzeros into equal chunks whatever rows they belong to (uneven rows:
 * many empty rows, or a share of the nonzeros in rows of more than 128); the list of non-empty rows that the second
 * form needs is built on the first SpMM call, in stream order, and so is the order of the rows by length that SpMM
 * uses when A has so few columns that a slice of B is kept in shared memory.
 * When the row statistics select the row-direct SpMV kernel, the first b200sp_spmv / spmv_csr call with a given
 * col_idx additionally samples how local the columns are (one small kernel and one synchronisation of the stream)
 * and falls back to the merge-tile kernel for matrices with scattered columns.
 * It takes one block of a few bytes per tile from the library's pool, in the order of `stream`, and
 * synchronises `stream` once.  A plan may be used from one stream at a time.  b200sp_plan_destroy
 * synchronises the plan's device before it returns the block. */
int b200sp_plan_create(b200sp_plan** out, int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, void* stream);
int b200sp_plan_destroy(b200sp_plan* plan);
int b200sp_plan_info(const b200sp_plan* plan, b200sp_plan_info_t* out); /* `out` is a host pointer */

/* Same operations as spmv_csr / spmm_csr with an explicit plan (m, n, nnz, row_ptr come from it). */
int b200sp_spmv(b200sp_plan* plan, const int32_t* col_idx, const void* vals, const void* x, void* y,
                float alpha, float beta, int dtype, void* stream);
int b200sp_spmm(b200sp_plan* plan, int64_t k, const int32_t* col_idx, const void* vals, const void* B, void* Y,
                float alpha, float beta, int dtype, void* stream);

/* ---- COO, CSC and ELL front ends -------------------------------------------------------------------
 * The other sparse formats of the paper's benchmark (Appendix C, Table 6): tasks 8 / 9 "SpMV / SpMM COO"
 * (values, row_indices, col_indices, each nnz long) and tasks 14 / 15 "SpMV / SpMM ELL" (values and
 * col_ids of size rows x max_nnz_per_row, padding positions marked with -1).  Same operations, scalars,
 * dtypes, alignment and stream conventions as spmv_csr / spmm_csr.
 *
 * COO: entries must be sorted by row (row_idx non-decreasing; columns within a row in any order).  The
 * first call for a given (device, row_idx, m, n, nnz) derives the row offsets on the device, checks the
 * order (synchronises the stream once), caches them, and then runs the CSR kernels; unsorted or
 * out-of-range row indices return B200SP_ERR_UNSUPPORTED.  b200sp_cache_clear drops the cached offsets.
 *
 * CSC (tasks 10 / 11: values, row_indices, col_offsets of cols + 1 entries): the first call for a given
 * (device, col_ptr, row_idx, m, n, nnz) builds the row-major order of the entries on the device (row counts, an
 * exclusive scan, placement, and a sort of every row's entries by their CSC position, so that a row's entries are
 * added in ascending column order on every run) and caches it together with a scratch array of nnz values; it
 * synchronises the stream twice.  Every call then permutes vals into that order with one kernel and runs the
 * CSR kernels.  Inconsistent col_ptr / row_idx return B200SP_ERR_BAD_CSR.  Calls that share a cached pattern
 * must not overlap on the GPU.
 *
 * ELL: row-major, row i occupies entries [i*width, (i+1)*width) of col_ids and vals; an entry is padding
 * when its col_id is negative (its value is ignored, whatever it holds).  m * width < 2^31.  No plan, no
 * cache, no synchronisation. */
int spmv_coo(int64_t m, int64_t n, int64_t nnz, const int32_t* row_idx, const int32_t* col_idx, const void* vals,
             const void* x, void* y, float alpha, float beta, int dtype, void* stream);
int spmm_coo(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_idx, const int32_t* col_idx, const void* vals,
             const void* B, void* Y, float alpha, float beta, int dtype, void* stream);
int spmv_csc(int64_t m, int64_t n, int64_t nnz, const int32_t* col_ptr, const int32_t* row_idx, const void* vals,
             const void* x, void* y, float alpha, float beta, int dtype, void* stream);
int spmm_csc(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* col_ptr, const int32_t* row_idx, const void* vals,
             const void* B, void* Y, float alpha, float beta, int dtype, void* stream);
int spmv_ell(int64_t m, int64_t n, int64_t width, const int32_t* col_ids, const void* vals, const void* x, void* y,
             float alpha, float beta, int dtype, void* stream);
int spmm_ell(int64_t m, int64_t n, int64_t width, int64_t k, const int32_t* col_ids, const void* vals, const void* B, void* Y,
             float alpha, float beta, int dtype, void* stream);

/* ---- SpMV without any allocation ---------------------------------------------------------------
 * (The paper has no counterpart for this entry point; it exists for callers of this library.)
 *
 * Some callers may not allocate device memory at all: code running inside a region where the
 * allocator is off limits (a real-time or safety-certified loop whose memory was fixed at start-up,
 * a plugin that must not touch its host's memory pools, a caller that has already handed every byte
 * of the GPU to its own arena).  For them spmv_csr_noalloc computes the same y = alpha*A*x + beta*y
 * as spmv_csr with the merge-tile kernel and its carry fix-up, but takes the scratch those kernels
 * need (tile split points, carries, tails) from a fixed array compiled into the library instead of a
 * plan: it calls no cudaMalloc / cudaFree and no allocating routine, builds no plan, caches nothing
 * and never synchronises.  All pointers are device pointers, as for spmv_csr.
 *
 *  - Limit: m + nnz <= b200sp_noalloc_max_items() (268,435,456; the array is about 0.75 MB, held by
 *    every GPU that loads the library until the process exits).  Larger problems are refused with
 *    B200SP_ERR_TOO_LARGE and nothing is launched.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current).  Make that first call before starting any stream capture.
 *  - Every call uses the same array and finds the previous call's contents in it; each call rewrites
 *    all the entries it later reads, so nothing needs clearing.  Two calls whose kernels overlap on the
 *    GPU (different streams, no ordering between them) race on the array: order them. */
int spmv_csr_noalloc(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx,
                     const void* vals, const void* x, void* y, float alpha, float beta, int dtype, void* stream);
int64_t b200sp_noalloc_max_items(void);   /* largest m + nnz that spmv_csr_noalloc accepts */

/* ---- host-buffer calls -----------------------------------------------------------------------
 * Same operations with every array in HOST memory (pinned memory makes the copies asynchronous and
 * faster, pageable memory works).  Each call takes device buffers from the library's stream-ordered pool,
 * copies the inputs in, plans, runs the kernels, copies y / Y back and synchronises `stream` before returning.
 * The plan is cached under the HOST address of row_ptr and (m, n, nnz) like the plans of the device entry points, with
 * the same rule: the contents of row_ptr must not change while it is cached (b200sp_cache_drop(row_ptr) forgets it). */
int spmv_csr_host(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx,
                  const void* vals, const void* x, void* y, float alpha, float beta, int dtype, void* stream);
int spmm_csr_host(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr, const int32_t* col_idx,
                  const void* vals, const void* B, void* Y, float alpha, float beta, int dtype, void* stream);
/* The matrix (row_ptr, col_idx, vals) is resident on the DEVICE, x and y are HOST buffers: copies x (and y when
 * beta != 0) in, runs spmv_csr with its cached plan, copies y back and synchronises `stream`.  This is one step of
 * an iterative method whose matrix stays on the GPU. */
int spmv_csr_vec_host(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, const void* vals,
                      const void* x_host, void* y_host, float alpha, float beta, int dtype, void* stream);

/* ---- checking and housekeeping ---------------------------------------------------------------
 * b200sp_validate_csr checks on the device that row_ptr[0] = 0, row_ptr[m] = nnz, row_ptr is
 * non-decreasing and every column index lies in [0, n); it synchronises the stream and returns
 * B200SP_ERR_BAD_CSR if any check fails. */
int b200sp_validate_csr(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, void* stream);

void b200sp_cache_clear(void);                 /* destroys every plan cached by the one-shot calls, trims the library's memory pools and
                                                  releases the L2 set aside for access-policy windows (option "x_l2_window") */
/* Forgets what the one-shot entry points cached under this address on the current device: the plan keyed on a row_ptr
 * (device address, or host address for the *_host calls), the row offsets keyed on a COO row_idx, the transpose plan
 * keyed on a CSC col_ptr.  Synchronises the device if anything was dropped.  Unknown addresses are not an error. */
int b200sp_cache_drop(const void* key_ptr);
const char* b200sp_status_string(int status);  /* static string, never NULL */
const char* b200sp_last_cuda_error(void);      /* message of this thread's last failing CUDA call, "" if none */
int b200sp_version(void);                      /* major * 10000 + minor * 100 + patch */
/* 1 if the library was built with -DB200SP_BOUNDS_CHECK (libb200sp_check.so): every SpMV / SpMM call then validates the matrix
 * on the device as b200sp_validate_csr does (one more kernel and one synchronisation of the stream per call) and returns
 * B200SP_ERR_BAD_CSR, launching nothing else, if row_ptr or a column index is out of range.  0 for the ordinary build. */
int b200sp_checked_build(void);

/* Synchronises `stream`, then reports whether any kernel of this library on the current device gave up
 * on a bounded wait (a staged copy that never signalled its barrier): B200SP_ERR_TIMEOUT if so (the
 * flag is cleared), else B200SP_OK.  The kernels never spin without a limit; a result produced by a
 * launch that timed out is incomplete. */
int b200sp_check(void* stream);

/* Naive baselines: one thread per row (SpMV) / per output entry (SpMM), scalar loads, sequential sums.
 * They play the role of the unoptimised baseline kernel that the paper's performance score (Section 3.3,
 * Eq. 1-2: speed-up over the baseline, weighted by the baseline's complexity T(N)) is measured against.
 * Same arguments and conventions as spmv_csr / spmm_csr, no plan, no alignment requirement; never used by them. */
int b200sp_spmv_naive(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, const void* vals,
                      const void* x, void* y, float alpha, float beta, int dtype, void* stream);
int b200sp_spmm_naive(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr, const int32_t* col_idx, const void* vals,
                      const void* B, void* Y, float alpha, float beta, int dtype, void* stream);

/* Number of kernels this library has launched from this process so far (all entry points). */
int64_t b200sp_launch_count(void);

/* Tuning switches, test switches and measurement probes live in b200sp_tuning.h: they are not part of the contract above. */

#ifdef __cplusplus
}
#endif
#endif /* B200SP_H_ */
