// CSR SpMV kernels: y = alpha * A * x + beta * y  (paper, Appendix C, Table 6, task 12, with alpha/beta).
//
// merge-tile kernel: the work list is the merge of row-end markers and nonzeros; every CTA takes
// ITEMS consecutive merge items, so a tile is bounded both in nonzeros and in rows whatever the
// row-length distribution.  Inside a tile:
//   phase 1  the tile's nonzeros are streamed in flat order with 128-bit loads, x is gathered
//            through the read-only path and the products go to shared memory;
//   phase 2  (short rows) one thread per row adds its products sequentially;
//   phase 3  (long rows, and the unfinished row at the tile's end) one warp per segment adds
//            lane-strided partial sums and combines them with __shfl_xor.
// A row cut by a tile boundary is not written by the tiles: each tile stores the partial sum of its
// unfinished last row in carry[t], the tile that holds the row's end stores its part in tail[t], and
// the fix-up kernel adds these in tile order and applies the epilogue once.  No atomics on floats.
// The merge list's rows are either the matrix's own rows (row_id == nullptr) or, for matrices with many empty rows, the rows that
// have nonzeros (m of them, row_ptr their m + 1 offsets, row_id[r] the matrix row of list row r).
#pragma once
#include "common.cuh"

namespace b200sp {

__device__ __forceinline__ int pad_index(int i) { return i + (i >> 5); }  // one spare word per 32: breaks power-of-two strides

template <typename T, int ITEMS, int THREADS, int SHORT_MAX>
__global__ void __launch_bounds__(THREADS)
spmv_merge_tile_kernel(int m, int nnz, const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                       const T* __restrict__ vals, const T* __restrict__ x, T* __restrict__ y, float alpha, float beta,
                       const int* __restrict__ split_row, float* __restrict__ carry, float* __restrict__ tail,
                       const int* __restrict__ row_id) {
  constexpr int G = 4;                      // nonzeros per vector load
  constexpr int PROD_N = ITEMS + 2 * G;     // products of one tile, counted from the aligned start
  constexpr int MAX_LONG = ITEMS / (SHORT_MAX + 1) + 2;
  constexpr int WARPS = THREADS / 32;
  constexpr int PROD_SIZE = PROD_N + PROD_N / 32 + 1 + 8;
  __shared__ float prod[PROD_SIZE];         // products from the front; the tile's row bounds (as ints) from the back: rows + nonzeros <= ITEMS, so they never meet
  __shared__ int long_rows[MAX_LONG];       // row of each long segment; -row-1 when the row began in an earlier tile
  __shared__ int2 long_span[MAX_LONG];      // its products: local [first, last)
  __shared__ int n_long;

  grid_dependency_wait();
  const int tid = threadIdx.x;
  const int t = blockIdx.x;
  const long long total = (long long)m + nnz;
  const long long d0 = (long long)t * ITEMS;
  const long long d1 = min(d0 + ITEMS, total);
  const int r0 = split_row[t], r1 = split_row[t + 1];
  const int p0 = (int)(d0 - r0), p1 = (int)(d1 - r1);
  const int a0 = p0 & ~(G - 1);
  if (tid == 0) n_long = 0;
  const int carry_start = r1 < m ? __ldg(row_ptr + r1) : 0;   // start of the unfinished last row, needed in phase 3: requested early
  // row_ptr[r0 .. r1] into the unused tail of prod (entry j at PROD_SIZE - 1 - j): phase 2 then needs no global load,
  // which is what rows without nonzeros would otherwise spend their time waiting for
  int* const bound_s = reinterpret_cast<int*>(prod) + (PROD_SIZE - 1);
#pragma unroll 4
  for (int j = tid; j <= r1 - r0; j += THREADS) bound_s[-j] = __ldg(row_ptr + r0 + j);

  // ---- phase 1: products of nonzeros [p0, p1) in flat order
  const int nq = (p1 - a0 + G - 1) / G;
  constexpr int U = 2;                      // vector loads in flight per thread: 32 registers, so the CTAs per SM are set by the carveout (measured on the power-law workload: 150 us against 157 us with four)
  for (int qb = 0; qb < nq; qb += THREADS * U) {
    int c[U][G];
    float v[U][G];
    bool ok[U][G];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int q = qb + u * THREADS + tid;
      const int base = a0 + q * G;
      if (q < nq && base >= p0 && base + G <= p1) {
        const int4 cc = ld_stream_i4(col_idx + base);
        c[u][0] = cc.x; c[u][1] = cc.y; c[u][2] = cc.z; c[u][3] = cc.w;
        ld_stream_vals4(vals + base, v[u]);
#pragma unroll
        for (int j = 0; j < G; ++j) ok[u][j] = true;
      } else {
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const int p = base + j;
          ok[u][j] = (q < nq) && p >= p0 && p < p1;
          c[u][j] = ok[u][j] ? ld_stream_i1(col_idx + p) : 0;
          v[u][j] = ok[u][j] ? ld_stream_val1(vals + p) : 0.0f;
        }
      }
    }
    float xv[U][G];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int j = 0; j < G; ++j) xv[u][j] = ok[u][j] ? ld_gather(x + c[u][j]) : 0.0f;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int q = qb + u * THREADS + tid;
      if (q < nq) {
#pragma unroll
        for (int j = 0; j < G; ++j) prod[pad_index(q * G + j)] = v[u][j] * xv[u][j];
      }
    }
  }
  __syncthreads();

  // ---- phase 2: rows whose end lies in this tile, one thread per row
  for (int r = r0 + tid; r < r1; r += THREADS) {
    const int rs = bound_s[r0 - r], re = bound_s[r0 - r - 1];
    const int s = max(rs, p0);
    const int len = re - s;
    if (len <= SHORT_MAX) {
      float acc = 0.0f;
      for (int q = s - a0; q < re - a0; ++q) acc += prod[pad_index(q)];
      if (rs < p0) tail[t] = acc;            // row began in an earlier tile: completed by the fix-up kernel
      else epilogue_store(y, row_id ? (long long)__ldg(row_id + r) : (long long)r, acc, alpha, beta);
    } else {
      const int slot = atomicAdd(&n_long, 1);  // order of the list does not affect any value
      long_rows[slot] = rs < p0 ? -r - 1 : r;
      long_span[slot] = make_int2(s - a0, re - a0);
    }
  }
  __syncthreads();

  // ---- phase 3: long segments, one warp each; then the unfinished row at the tile's end
  const int warp = tid >> 5, lane = tid & 31;
  const int nl = n_long;
  for (int i = warp; i < nl; i += WARPS) {
    const int r = long_rows[i];
    const int2 span = long_span[i];
    float acc = 0.0f;
    for (int q = span.x + lane; q < span.y; q += 32) acc += prod[pad_index(q)];
    acc = warp_sum(acc);
    if (lane == 0) {
      if (r < 0) tail[t] = acc;
      else epilogue_store(y, row_id ? (long long)__ldg(row_id + r) : (long long)r, acc, alpha, beta);
    }
  }
  if (warp == WARPS - 1) {
    float acc = 0.0f;
    if (r1 < m) {
      const int s = max(carry_start, p0);
      for (int q = s - a0 + lane; q < p1 - a0; q += 32) acc += prod[pad_index(q)];
      acc = warp_sum(acc);
    }
    if (lane == 0) carry[t] = acc;
  }
}

// Completes the rows that a tile boundary cut: tile t owns such a row when its first row began
// before the tile's first nonzero.  The row's value is carry[first] + ... + carry[t-1] + tail[t],
// added in that fixed order, then the epilogue is applied once.
template <typename T, int ITEMS>
__global__ void __launch_bounds__(128)
spmv_carry_fixup_kernel(int tiles, const int* __restrict__ row_ptr, const int* __restrict__ split_row,
                        const float* __restrict__ carry, const float* __restrict__ tail, T* __restrict__ y, float alpha, float beta,
                        const int* __restrict__ row_id) {
  grid_dependency_wait();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < 1 || t >= tiles) return;
  const int r0 = split_row[t];
  if (r0 >= split_row[t + 1]) return;                 // the tile holds no row end
  const long long p0 = (long long)t * ITEMS - r0;
  if ((long long)row_ptr[r0] >= p0) return;           // its first row starts inside the tile
  int tf = t - 1;
  while (tf > 0 && split_row[tf] == r0) --tf;         // earlier tiles that lie entirely inside row r0
  float acc = 0.0f;
  for (int u = tf; u < t; ++u) acc += carry[u];
  acc += tail[t];
  epilogue_store(y, row_id ? (long long)row_id[r0] : (long long)r0, acc, alpha, beta);
}

// y[i] = beta * y[i] for the rows without nonzeros (beta != 0): the pass that goes with a merge list of non-empty rows.
template <typename T>
__global__ void __launch_bounds__(256) scale_empty_rows_kernel(long long m, const int* __restrict__ row_ptr, T* __restrict__ y, float beta) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < m; i += (long long)gridDim.x * blockDim.x)
    if (row_ptr[i] == row_ptr[i + 1]) epilogue_store(y, i, 0.0f, 0.0f, beta);
}

// y = beta * y (or 0 when beta == 0): used when alpha == 0 or the matrix has no nonzeros.
template <typename T>
__global__ void __launch_bounds__(256) scale_kernel(long long count, T* __restrict__ y, float beta) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x)
    epilogue_store(y, i, 0.0f, 0.0f, beta);
}

}  // namespace b200sp
