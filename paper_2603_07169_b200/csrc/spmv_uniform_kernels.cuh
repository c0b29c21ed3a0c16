// Sub-warp-per-row CSR SpMV kernel for matrices whose rows all have the same length L = 4 * LPR,
// LPR a power of two (plan: min row length == max row length):
// y = alpha * A * x + beta * y  (paper, Appendix C, Table 6, task 12, with alpha/beta).
//
// With equal rows, row r starts at nonzero r * L, so row_ptr need not be read and every group of
// four nonzeros is 16-byte aligned: each lane streams one int4 of col_idx and four vals with
// 128-bit coalesced loads, gathers four x entries through the read-only path, and LPR adjacent lanes
// combine their partial sums with __shfl_xor.  No shared memory is used, so the whole unified cache
// serves as L1 for the gather (its capacity bounds the number of misses in flight, which is what
// limits a gather over a vector much larger than L1).  UNROLL independent groups per thread keep
// 4 * UNROLL gathers in flight.  The reduction order is fixed, so results are bit-reproducible.
#pragma once
#include "common.cuh"

namespace b200sp {

template <typename T, int LPR, int UNROLL, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmv_uniform_vec_kernel(long long quads, const int* __restrict__ col_idx, const T* __restrict__ vals,
                        const T* __restrict__ x, T* __restrict__ y, float alpha, float beta) {
  grid_dependency_wait();
  const long long stride = (long long)gridDim.x * THREADS;
  long long g = (long long)blockIdx.x * THREADS + threadIdx.x;
  // every lane of a warp runs the same number of iterations: quads is a multiple of LPR and warps start on multiples of 32
  for (; g < quads; g += stride * UNROLL) {
    int4 c[UNROLL];
    float v[UNROLL][4];
    float yold[UNROLL];
    bool ok[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const long long q = g + (long long)u * stride;
      ok[u] = q < quads;
      yold[u] = 0.0f;
      if (ok[u]) {
        c[u] = ld_stream_i4(col_idx + q * 4);
        ld_stream_vals4(vals + q * 4, v[u]);
        if (beta != 0.0f && (q & (LPR - 1)) == 0) yold[u] = to_f32(y[q / LPR]);   // asked for now: its latency overlaps the gathers
      }
    }
    float part[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      part[u] = 0.0f;
      if (ok[u]) {
        const float x0 = ld_gather(x + c[u].x), x1 = ld_gather(x + c[u].y), x2 = ld_gather(x + c[u].z), x3 = ld_gather(x + c[u].w);
        part[u] = fmaf(v[u][3], x3, fmaf(v[u][2], x2, fmaf(v[u][1], x1, v[u][0] * x0)));
      }
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const long long q = g + (long long)u * stride;
      // the lanes of one row either all pass `ok` or all fail it, and whole warps stay converged here
      float s = part[u];
#pragma unroll
      for (int o = 1; o < LPR; o <<= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
      if (ok[u] && (q & (LPR - 1)) == 0) {
        float r = alpha * s;
        if (beta != 0.0f) r += beta * yold[u];
        store_elem(y + q / LPR, r);
      }
    }
  }
}

}  // namespace b200sp

namespace b200sp {

// Sub-warp-per-row kernel for small problems (the launch-latency regime, e.g. the paper's own SpMV sizes:
// 2^10..2^15 rows x 2048 columns at 1 % density).  LPR adjacent lanes own one row and stride over its
// nonzeros, partial sums are combined with __shfl_xor, lane 0 of the group applies the epilogue.  No plan
// scratch and no shared memory: the dependent chain is row_ptr -> (col_idx, vals) -> x -> store, and the
// grid has one group per row so that even a few thousand rows spread over all SMs.
template <typename T, int LPR, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmv_subwarp_kernel(int m, const int* __restrict__ row_ptr, const int* __restrict__ col_idx, const T* __restrict__ vals,
                    const T* __restrict__ x, T* __restrict__ y, float alpha, float beta) {
  grid_dependency_wait();
  const long long gid = (long long)blockIdx.x * THREADS + threadIdx.x;
  const long long row = gid / LPR;
  const int sub = (int)(gid % LPR);
  int rs = 0, re = 0;
  if (row < m) { rs = __ldg(row_ptr + row); re = __ldg(row_ptr + row + 1); }
  float acc = 0.0f;
  int p = rs + sub;
  for (; p + LPR < re; p += 2 * LPR) {   // two independent gathers per lane and trip
    const int c0 = __ldg(col_idx + p), c1 = __ldg(col_idx + p + LPR);
    const float v0 = to_f32(__ldg(vals + p)), v1 = to_f32(__ldg(vals + p + LPR));
    const float x0 = ld_gather(x + c0), x1 = ld_gather(x + c1);
    acc = fmaf(v1, x1, fmaf(v0, x0, acc));
  }
  if (p < re) acc = fmaf(to_f32(__ldg(vals + p)), ld_gather(x + __ldg(col_idx + p)), acc);
#pragma unroll
  for (int o = 1; o < LPR; o <<= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if (row < m && sub == 0) epilogue_store(y, row, acc, alpha, beta);
}

// Reference-quality baseline: one thread per row, scalar loads, sequential sum.  This is the "naive kernel"
// that the paper's speed-up metric (Section 3.3, Eq. 1-2) is measured against; it is not used by spmv_csr.
template <typename T>
__global__ void __launch_bounds__(256)
spmv_naive_kernel(int m, const int* __restrict__ row_ptr, const int* __restrict__ col_idx, const T* __restrict__ vals,
                  const T* __restrict__ x, T* __restrict__ y, float alpha, float beta) {
  const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= m) return;
  float acc = 0.0f;
  for (int p = row_ptr[row]; p < row_ptr[row + 1]; ++p) acc += to_f32(vals[p]) * to_f32(x[col_idx[p]]);
  epilogue_store(y, row, acc, alpha, beta);
}

// Naive SpMM baseline: one thread per output entry Y[i, c].
template <typename T>
__global__ void __launch_bounds__(256)
spmm_naive_kernel(long long m, int k, const int* __restrict__ row_ptr, const int* __restrict__ col_idx, const T* __restrict__ vals,
                  const T* __restrict__ B, T* __restrict__ Y, float alpha, float beta) {
  const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= m * k) return;
  const long long row = id / k;
  const int c = (int)(id - row * k);
  float acc = 0.0f;
  for (int p = row_ptr[row]; p < row_ptr[row + 1]; ++p) acc += to_f32(vals[p]) * to_f32(B[(long long)col_idx[p] * k + c]);
  epilogue_store(Y, id, acc, alpha, beta);
}

}  // namespace b200sp
