// COO and ELL front ends (paper, Appendix C, Table 6: tasks 8 / 9 SpMV / SpMM COO, tasks 14 / 15 SpMV / SpMM ELL).
//
// COO (values, row_indices, col_indices) with entries sorted by row is CSR without the offsets: a device
// pass finds each row's first entry by binary search, after which the CSR kernels run unchanged.
// ELL (values and col_ids of size rows x width, row-major, padding marked by col_id < 0) is CSR with the
// implicit offsets i * width; its kernels skip the padded entries.
#pragma once
#include "common.cuh"
#include "spmm_kernels.cuh"

namespace b200sp {

// row_ptr[r] = first position p with row_idx[p] >= r, for r = 0..m; flags unsorted or out-of-range row indices.
__global__ void __launch_bounds__(256) coo_row_ptr_kernel(const int* __restrict__ row_idx, int nnz, int m, int* __restrict__ row_ptr,
                                                          int* __restrict__ bad) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (long long r = i0; r <= m; r += stride) {
    int lo = 0, hi = nnz;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (row_idx[mid] < r) lo = mid + 1; else hi = mid; }
    row_ptr[r] = lo;
  }
  int b = 0;
  for (long long p = i0; p < nnz; p += stride) {
    const int r = row_idx[p];
    if (r < 0 || r >= m) b = 1;
    if (p + 1 < nnz && row_idx[p + 1] < r) b = 1;
  }
  if (b) atomicOr(bad, 1);
}

// CSC front end, per call: values permuted into the row-major order that the transpose plan computed.
template <typename T>
__global__ void __launch_bounds__(256) csc_permute_vals_kernel(long long nnz, const int* __restrict__ perm, const T* __restrict__ vals,
                                                               T* __restrict__ vals_t) {
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < nnz; q += (long long)gridDim.x * blockDim.x)
    vals_t[q] = vals[perm[q]];
}

// ELL SpMV: LPR adjacent lanes own one row and stride over its `width` slots, VECW slots per load.
template <typename T, int LPR, int VECW, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmv_ell_kernel(int m, int width, const int* __restrict__ col_ids, const T* __restrict__ vals, const T* __restrict__ x,
                T* __restrict__ y, float alpha, float beta) {
  grid_dependency_wait();
  const long long gid = (long long)blockIdx.x * THREADS + threadIdx.x;
  const long long row = gid / LPR;
  const int sub = (int)(gid % LPR);
  float acc = 0.0f, tot = 0.0f;   // acc: at most kChainBlock products in one chain, then folded into tot
  int trips = 0;
  if (row < m) {
    const long long base = row * width;
    if (VECW == 4) {
      int j = sub * 4;
      for (; j + LPR * 4 < width; j += 2 * LPR * 4) {   // two independent groups of four per trip
        if (++trips > kChainBlock / 8) { trips = 1; tot += acc; acc = 0.0f; }
        const int4 c0 = ld_stream_i4(col_ids + base + j), c1 = ld_stream_i4(col_ids + base + j + LPR * 4);
        float v0[4], v1[4];
        ld_stream_vals4(vals + base + j, v0);
        ld_stream_vals4(vals + base + j + LPR * 4, v1);
        const int cc[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
        float xv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) xv[u] = cc[u] >= 0 ? ld_gather(x + cc[u]) : 0.0f;
#pragma unroll
        for (int u = 0; u < 4; ++u) acc = fmaf(cc[u] >= 0 ? v0[u] : 0.0f, xv[u], acc);
#pragma unroll
        for (int u = 0; u < 4; ++u) acc = fmaf(cc[4 + u] >= 0 ? v1[u] : 0.0f, xv[4 + u], acc);
      }
      if (j < width) {
        const int4 c0 = ld_stream_i4(col_ids + base + j);
        float v0[4];
        ld_stream_vals4(vals + base + j, v0);
        const int cc[4] = {c0.x, c0.y, c0.z, c0.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) if (cc[u] >= 0) acc = fmaf(v0[u], ld_gather(x + cc[u]), acc);
      }
    } else {
      for (int j = sub; j < width; j += LPR) {
        if (++trips > kChainBlock) { trips = 1; tot += acc; acc = 0.0f; }
        const int c = ld_stream_i1(col_ids + base + j);
        if (c >= 0) acc = fmaf(ld_stream_val1(vals + base + j), ld_gather(x + c), acc);
      }
    }
  }
  acc += tot;
#pragma unroll
  for (int o = 1; o < LPR; o <<= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if (row < m && sub == 0) epilogue_store(y, row, acc, alpha, beta);
}

// ELL SpMM, k-sliced like spmm_slice_kernel: eight lanes per row, 128 bytes of B per nonzero and slice.
template <typename T, int VEC, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmm_ell_slice_kernel(int m, int k, int width, int row_blocks, const int* __restrict__ col_ids, const T* __restrict__ vals,
                      const T* __restrict__ B, T* __restrict__ Y, float alpha, float beta) {
  constexpr int LANES = 8, GROUPS = THREADS / LANES, KS = LANES * VEC;
  typedef typename RawVec<T, VEC>::type raw_t;
  const int slice = blockIdx.x / row_blocks, rb = blockIdx.x - slice * row_blocks;
  const int g = threadIdx.x / LANES, l8 = threadIdx.x % LANES;
  const long long row = (long long)rb * GROUPS + g;
  if (row >= m) return;
  const int col0 = slice * KS + l8 * VEC;
  if (col0 >= k) return;
  const T* Bc = B + col0;
  const long long base = row * width;
  float acc[VEC], tot[VEC];   // blocks of at most kChainBlock products, block sums in a second chain
#pragma unroll
  for (int j = 0; j < VEC; ++j) { acc[j] = 0.0f; tot[j] = 0.0f; }
  for (int j = 0; j < width; ++j) {
    if (j > 0 && j % kChainBlock == 0) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) { tot[i] += acc[i]; acc[i] = 0.0f; }
    }
    const int c = __ldg(col_ids + base + j);
    if (c >= 0) {
      const raw_t b = RawVec<T, VEC>::ld(Bc + (long long)c * k);
      RawVec<T, VEC>::fma(b, to_f32(__ldg(vals + base + j)), acc);
    }
  }
#pragma unroll
  for (int i = 0; i < VEC; ++i) acc[i] += tot[i];
  T* yp = Y + row * k + col0;
  float out[VEC];
  if (beta != 0.0f) {
    float old[VEC];
    VecLoad<T, VEC>::ld_plain(yp, old);
#pragma unroll
    for (int j = 0; j < VEC; ++j) out[j] = alpha * acc[j] + beta * old[j];
  } else {
#pragma unroll
    for (int j = 0; j < VEC; ++j) out[j] = alpha * acc[j];
  }
  VecLoad<T, VEC>::st(yp, out);
}

// ELL SpMM for any k: one thread per output entry (used when k is not a multiple of the vector width).
template <typename T>
__global__ void __launch_bounds__(256)
spmm_ell_entry_kernel(long long m, int k, int width, const int* __restrict__ col_ids, const T* __restrict__ vals,
                      const T* __restrict__ B, T* __restrict__ Y, float alpha, float beta) {
  const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= m * k) return;
  const long long row = id / k;
  const int c = (int)(id - row * k);
  float acc = 0.0f, tot = 0.0f;
  for (int j = 0; j < width; ++j) {
    if (j > 0 && j % kChainBlock == 0) { tot += acc; acc = 0.0f; }
    const int col = col_ids[row * width + j];
    if (col >= 0) acc = fmaf(to_f32(vals[row * width + j]), to_f32(B[(long long)col * k + c]), acc);
  }
  epilogue_store(Y, id, acc + tot, alpha, beta);
}

}  // namespace b200sp
