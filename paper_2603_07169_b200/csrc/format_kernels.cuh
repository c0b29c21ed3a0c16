// COO and ELL front ends (paper, Appendix C, Table 6: tasks 8 / 9 SpMV / SpMM COO, tasks 14 / 15 SpMV / SpMM ELL).
//
// COO (values, row_indices, col_indices) with entries sorted by row is CSR without the offsets: a device
// pass finds each row's first entry by binary search, after which the CSR kernels run unchanged.
// ELL (values and col_ids of size rows x width, row-major, padding marked by col_id < 0) is CSR with the
// implicit offsets i * width; its kernels skip the padded entries.
#pragma once
#include "common.cuh"
#include "plan_kernels.cuh"
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

// ---- CSC front end: the transpose plan, built on the device ----
// The row-major order of a CSC pattern: entry q of the row-major list is CSC entry perm[q], rows ascending and, inside a row,
// CSC positions ascending (= columns ascending, duplicates in their stored order), so that a row's sum is added in the same
// order on every run.  Steps: check the pattern; count the entries of each row (integer atomics: the counts do not depend on
// scheduling); exclusive scan -> row offsets; place every entry in its row's range at a slot claimed with an integer atomic
// (the order inside a row is arbitrary at this point); sort each row's range by CSC position (which makes it unique); look up each
// entry's column in col_ptr.

__global__ void __launch_bounds__(256) csc_check_kernel(const int* __restrict__ col_ptr, const int* __restrict__ row_idx, int m, int n, int nnz,
                                                        int* __restrict__ bad) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  int b = 0;
  if (i0 == 0 && (col_ptr[0] != 0 || col_ptr[n] != nnz)) b = 1;
  for (long long j = i0; j < n; j += stride) if (col_ptr[j + 1] < col_ptr[j]) b = 1;
  for (long long p = i0; p < nnz; p += stride) { const int r = row_idx[p]; if (r < 0 || r >= m) b = 1; }
  if (b) atomicOr(bad, 1);
}

__global__ void __launch_bounds__(256) csc_count_rows_kernel(const int* __restrict__ row_idx, long long nnz, int* __restrict__ count) {
  for (long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x; p < nnz; p += (long long)gridDim.x * blockDim.x)
    atomicAdd(count + row_idx[p], 1);
}

// Exclusive scan of an int array in three passes (blocks of kScanBlock entries): block sums; their exclusive scan by one CTA
// (plan_compact_scan_kernel); every block's own scan plus its offset.  out may alias in.  out[count] is not written.
constexpr int kScanBlock = 1024;

__global__ void __launch_bounds__(256) scan_block_sums_kernel(const int* __restrict__ in, long long count, int* __restrict__ block_sum) {
  __shared__ int s_sum;
  if (threadIdx.x == 0) s_sum = 0;
  __syncthreads();
  const long long base = (long long)blockIdx.x * kScanBlock;
  int c = 0;
  for (int j = threadIdx.x; j < kScanBlock; j += 256) if (base + j < count) c += in[base + j];
  atomicAdd(&s_sum, c);
  __syncthreads();
  if (threadIdx.x == 0) block_sum[blockIdx.x] = s_sum;
}

__global__ void __launch_bounds__(256) scan_apply_kernel(const int* in, long long count, const int* __restrict__ block_offset, int* out) {
  __shared__ int s_warp[8];
  const long long base = (long long)blockIdx.x * kScanBlock;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int running = block_offset[blockIdx.x];
  for (int j0 = 0; j0 < kScanBlock; j0 += 256) {
    const long long i = base + j0 + threadIdx.x;
    const int v = i < count ? in[i] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t; }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) { const int c = s_warp[w]; if (w < warp) before += c; total += c; }
    if (i < count) out[i] = running + before + incl - v;
    running += total;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(256) csc_place_kernel(const int* __restrict__ row_idx, long long nnz, const int* __restrict__ row_ptr_t,
                                                        int* __restrict__ fill, int* __restrict__ perm) {
  for (long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x; p < nnz; p += (long long)gridDim.x * blockDim.x) {
    const int r = row_idx[p];
    perm[row_ptr_t[r] + atomicAdd(fill + r, 1)] = (int)p;
  }
}

// Sorts every row's range of perm ascending.  A CTA owns 256 consecutive rows: rows of at most 32 entries are sorted by one
// thread each (insertion sort), longer rows one after another by the whole CTA with a bitonic network, in shared memory when the
// row fits (4096 entries), else in place in global memory.  Positions are distinct, so the result is unique.
__global__ void __launch_bounds__(256) csc_sort_rows_kernel(int m, const int* __restrict__ row_ptr_t, int* __restrict__ perm) {
  constexpr int CAP = 4096;
  __shared__ int buf[CAP];
  const long long row0 = (long long)blockIdx.x * 256;
  {
    const long long r = row0 + threadIdx.x;
    if (r < m) {
      const int s = row_ptr_t[r], e = row_ptr_t[r + 1];
      if (e - s <= 32) {
        for (int i = s + 1; i < e; ++i) {
          const int v = perm[i];
          int j = i - 1;
          while (j >= s && perm[j] > v) { perm[j + 1] = perm[j]; --j; }
          perm[j + 1] = v;
        }
      }
    }
  }
  for (int t = 0; t < 256; ++t) {
    const long long r = row0 + t;
    if (r >= m) break;
    const int s = row_ptr_t[r], len = row_ptr_t[r + 1] - s;
    if (len <= 32) continue;                       // uniform over the CTA: every thread reads the same bounds
    int pow2 = 64;
    while (pow2 < len) pow2 <<= 1;
    const bool in_smem = len <= CAP;
    __syncthreads();
    if (in_smem) {
      for (int i = threadIdx.x; i < len; i += 256) buf[i] = perm[s + i];
      __syncthreads();
    }
    int* const data = in_smem ? buf : perm + s;
    // bitonic network in the form whose comparisons all ascend (each merge starts with a mirrored step), so entries past len,
    // which would only ever be the larger partner, need not exist
    for (int size = 2; size <= pow2; size <<= 1) {
      const int half = size >> 1;
      for (int i = threadIdx.x; i < pow2 / 2; i += 256) {
        const int blk = i / half, off = i - blk * half;
        const int lo = blk * size + off, hi = blk * size + size - 1 - off;
        if (hi < len) { const int a = data[lo], b = data[hi]; if (a > b) { data[lo] = b; data[hi] = a; } }
      }
      __syncthreads();
      for (int stride = half >> 1; stride > 0; stride >>= 1) {
        for (int i = threadIdx.x; i < pow2 / 2; i += 256) {
          const int lo = 2 * i - (i & (stride - 1)), hi = lo + stride;
          if (hi < len) { const int a = data[lo], b = data[hi]; if (a > b) { data[lo] = b; data[hi] = a; } }
        }
        __syncthreads();
      }
    }
    if (in_smem) for (int i = threadIdx.x; i < len; i += 256) perm[s + i] = buf[i];
  }
}

// col_t[q] = the column of CSC entry perm[q]: the last j with col_ptr[j] <= perm[q].
__global__ void __launch_bounds__(256) csc_cols_kernel(long long nnz, int n, const int* __restrict__ col_ptr, const int* __restrict__ perm,
                                                       int* __restrict__ col_t) {
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < nnz; q += (long long)gridDim.x * blockDim.x) {
    const int p = perm[q];
    int lo = 0, hi = n;                             // first j with col_ptr[j] > p, minus one
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (col_ptr[mid + 1] <= p) lo = mid + 1; else hi = mid; }
    col_t[q] = lo;
  }
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
