// Plan pass (device side): row-length statistics and bins, merge-path split points, lists of medium and long rows.
#pragma once
#include "common.cuh"

namespace b200sp {

struct PlanStats {
  int min_len;
  int max_len;
  int bad;  // row_ptr not monotone (negative length seen)
  int pad;
  unsigned long long bin_rows[6];
  unsigned long long bin_nnz[6];
};

// Row-length bins: 0, 1-4, 5-32, 33-128, 129-1024, > 1024.
__device__ __forceinline__ int length_bin(int len) {
  return len == 0 ? 0 : len <= 4 ? 1 : len <= 32 ? 2 : len <= 128 ? 3 : len <= 1024 ? 4 : 5;
}

// One pass over row_ptr: min / max row length and the six length bins (rows, nnz per bin).
// Integer atomics only, so the result does not depend on scheduling.
__global__ void __launch_bounds__(256) plan_stats_kernel(const int* __restrict__ row_ptr, int m, PlanStats* st) {
  __shared__ unsigned long long s_rows[6], s_nnz[6];
  __shared__ int s_min, s_max, s_bad;
  if (threadIdx.x < 6) { s_rows[threadIdx.x] = 0; s_nnz[threadIdx.x] = 0; }
  if (threadIdx.x == 0) { s_min = 0x7FFFFFFF; s_max = 0; s_bad = 0; }
  __syncthreads();
  int lmin = 0x7FFFFFFF, lmax = 0, bad = 0;
  unsigned rows[6] = {0, 0, 0, 0, 0, 0};
  unsigned long long nz[6] = {0, 0, 0, 0, 0, 0};
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < m; i += (long long)gridDim.x * blockDim.x) {
    const int len = row_ptr[i + 1] - row_ptr[i];
    if (len < 0) { bad = 1; continue; }
    lmin = min(lmin, len); lmax = max(lmax, len);
    const int b = length_bin(len);
#pragma unroll
    for (int j = 0; j < 6; ++j) if (b == j) { rows[j]++; nz[j] += (unsigned)len; }
  }
  atomicMin(&s_min, lmin); atomicMax(&s_max, lmax); if (bad) atomicOr(&s_bad, 1);
#pragma unroll
  for (int j = 0; j < 6; ++j) if (rows[j]) { atomicAdd(&s_rows[j], (unsigned long long)rows[j]); atomicAdd(&s_nnz[j], nz[j]); }
  __syncthreads();
  if (threadIdx.x == 0) { atomicMin(&st->min_len, s_min); atomicMax(&st->max_len, s_max); if (s_bad) atomicOr(&st->bad, 1); }
  if (threadIdx.x < 6 && s_rows[threadIdx.x]) {
    atomicAdd(&st->bin_rows[threadIdx.x], s_rows[threadIdx.x]);
    atomicAdd(&st->bin_nnz[threadIdx.x], s_nnz[threadIdx.x]);
  }
}

// Merge-path split: the work list is the merge of the m row-end markers (row_ptr[1..m]) with the nnz
// nonzero positions 0..nnz-1; tile t starts at diagonal t * items.  split_row[t] = number of row ends
// consumed before that diagonal, so the tile's first nonzero is t * items - split_row[t].
__global__ void __launch_bounds__(256) plan_merge_split_kernel(const int* __restrict__ row_ptr, int m, int nnz, int items,
                                                               int tiles, int* __restrict__ split_row) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t > tiles) return;
  const long long total = (long long)m + nnz;
  long long d = (long long)t * items;
  if (d > total) d = total;
  int lo = (int)max(d - (long long)nnz, 0LL), hi = (int)min(d, (long long)m);
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if ((long long)row_ptr[mid + 1] <= d - mid - 1) lo = mid + 1; else hi = mid;
  }
  split_row[t] = lo;
}

// ---- list of the rows that have nonzeros (for matrices with many empty rows) ----
// Three passes: non-empty rows per block of kCompactBlock rows; an exclusive scan of the block counts by one CTA; then every
// block writes its rows' numbers and offsets at its place.  Integer work only; the order of the list is the row order.
constexpr int kCompactBlock = 1024;

__global__ void __launch_bounds__(256) plan_compact_count_kernel(const int* __restrict__ row_ptr, int m, int* __restrict__ block_count) {
  __shared__ int s_count;
  if (threadIdx.x == 0) s_count = 0;
  __syncthreads();
  const long long base = (long long)blockIdx.x * kCompactBlock;
  int c = 0;
  for (int j = threadIdx.x; j < kCompactBlock; j += 256) {
    const long long r = base + j;
    if (r < m && row_ptr[r + 1] > row_ptr[r]) ++c;
  }
  atomicAdd(&s_count, c);
  __syncthreads();
  if (threadIdx.x == 0) block_count[blockIdx.x] = s_count;
}

// block_count[b] <- sum of block_count[0 .. b-1]; block_count[blocks] <- total.  One CTA of 1024 threads.
__global__ void __launch_bounds__(1024) plan_compact_scan_kernel(int* __restrict__ block_count, int blocks) {
  __shared__ int s_warp[32];
  __shared__ int s_base;
  if (threadIdx.x == 0) s_base = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int b0 = 0; b0 < blocks; b0 += 1024) {
    const int b = b0 + threadIdx.x;
    const int v = b < blocks ? block_count[b] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t; }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = s_warp[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, w, o); if (lane >= o) w += t; }
      s_warp[lane] = w;
    }
    __syncthreads();
    const int before = s_base + (warp > 0 ? s_warp[warp - 1] : 0) + incl - v;
    if (b < blocks) block_count[b] = before;
    __syncthreads();
    if (threadIdx.x == 1023) s_base = before + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) block_count[blocks] = s_base;
}

__global__ void __launch_bounds__(256) plan_compact_write_kernel(const int* __restrict__ row_ptr, int m, int nnz, const int* __restrict__ block_offset,
                                                                 int* __restrict__ row_id, int* __restrict__ row_ptr_c) {
  __shared__ int s_warp[8];
  const long long base = (long long)blockIdx.x * kCompactBlock;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int out = block_offset[blockIdx.x];
  for (int j0 = 0; j0 < kCompactBlock; j0 += 256) {     // rows in order: four rounds of 256 consecutive rows
    const long long r = base + j0 + threadIdx.x;
    int rs = 0, flag = 0;
    if (r < m) { rs = row_ptr[r]; flag = row_ptr[r + 1] > rs ? 1 : 0; }
    const unsigned ballot = __ballot_sync(0xFFFFFFFFu, flag);
    if (lane == 0) s_warp[warp] = __popc(ballot);
    __syncthreads();
    int before = 0, round_total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) { const int c = s_warp[w]; if (w < warp) before += c; round_total += c; }
    if (flag) {
      const int slot = out + before + __popc(ballot & ((1u << lane) - 1u));
      row_id[slot] = (int)r;
      row_ptr_c[slot] = rs;
    }
    out += round_total;
    __syncthreads();
  }
  if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) row_ptr_c[out] = nnz;
}

// Tile starts of the nnz-balanced SpMM kernel: tile_row[t] = the row that holds nonzero t * tile_nnz, i.e. the first r with
// row_ptr[r + 1] > t * tile_nnz (rows without nonzeros are skipped over); m when t * tile_nnz >= nnz.
__global__ void __launch_bounds__(256) plan_nnz_tile_rows_kernel(const int* __restrict__ row_ptr, int m, int nnz, int tile_nnz, int tiles,
                                                                 int* __restrict__ tile_row) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t > tiles) return;
  const long long p = (long long)t * tile_nnz;
  if (p >= nnz) { tile_row[t] = m; return; }
  int lo = 0, hi = m - 1;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if ((long long)row_ptr[mid + 1] <= p) lo = mid + 1; else hi = mid;
  }
  tile_row[t] = lo;
}

// Rows of mid_thresh + 1 .. long_thresh nonzeros and rows longer than long_thresh, each appended to a list of its own
// (count[0], count[1]; the host sorts the lists, and their order only affects scheduling, never a value).
__global__ void __launch_bounds__(256) plan_row_lists_kernel(const int* __restrict__ row_ptr, int m, int mid_thresh, int long_thresh,
                                                             int mid_cap, int long_cap, int* __restrict__ mid_list,
                                                             int* __restrict__ long_list, int* __restrict__ count) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < m; i += (long long)gridDim.x * blockDim.x) {
    const int len = row_ptr[i + 1] - row_ptr[i];
    if (len > long_thresh) {
      const int slot = atomicAdd(count + 1, 1);
      if (slot < long_cap) long_list[slot] = (int)i;
    } else if (len > mid_thresh) {
      const int slot = atomicAdd(count, 1);
      if (slot < mid_cap) mid_list[slot] = (int)i;
    }
  }
}

// ---- processing order of the SpMM kernel that keeps a slice of B in shared memory --------------------------------
// That kernel gives a lane group one row at a time and a warp `gpw` rows per step, so a step lasts as long as its
// longest row, and lane groups whose rows differ in length by less than four still part ways in the last, partly filled
// group of four nonzeros.  The rows of at most kLongRow nonzeros are therefore sorted by their length (0 .. kLongRow),
// longest first, with a stable counting sort in three passes: per-block histograms
// (one warp per block of `rows_per_blk` consecutive rows), an exclusive scan of the (key, block) table, and a
// scatter in which a warp walks its rows in order, so that equal keys keep their row order.  Integer work only.
constexpr int kQuadKeys = 1024 + 1;   // kLongRow + 1

__device__ __forceinline__ int quad_key(int len) { return len > 1024 ? -1 : kQuadKeys - 1 - len; }

__global__ void __launch_bounds__(128) quad_order_hist_kernel(const int* __restrict__ row_ptr, int m, int rows_per_blk, int nblk,
                                                              int* __restrict__ hist) {
  __shared__ int s_hist[4][kQuadKeys];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blk = blockIdx.x * 4 + warp;
  for (int j = lane; j < kQuadKeys; j += 32) s_hist[warp][j] = 0;
  __syncwarp();
  if (blk < nblk) {
    const long long r0 = (long long)blk * rows_per_blk;
    const long long r1 = min((long long)m, r0 + rows_per_blk);
    for (long long r = r0 + lane; r < r1; r += 32) {
      const int key = quad_key(__ldg(row_ptr + r + 1) - __ldg(row_ptr + r));
      if (key >= 0) atomicAdd(&s_hist[warp][key], 1);
    }
    __syncwarp();
    for (int j = lane; j < kQuadKeys; j += 32) hist[(long long)j * nblk + blk] = s_hist[warp][j];
  }
}

// offset: the scanned table.  row_of / len_of: the sorted list (slots past its end are preset by the caller).
__global__ void __launch_bounds__(128) quad_order_scatter_kernel(const int* __restrict__ row_ptr, int m, int rows_per_blk, int nblk,
                                                                 const int* __restrict__ offset, int* __restrict__ row_of,
                                                                 int* __restrict__ len_of) {
  __shared__ int s_next[4][kQuadKeys];
  constexpr unsigned FULL = 0xFFFFFFFFu;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blk = blockIdx.x * 4 + warp;
  if (blk >= nblk) return;
  for (int j = lane; j < kQuadKeys; j += 32) s_next[warp][j] = offset[(long long)j * nblk + blk];
  __syncwarp();
  const long long r0 = (long long)blk * rows_per_blk;
  const long long r1 = min((long long)m, r0 + rows_per_blk);
  for (long long rb = r0; rb < r1; rb += 32) {
    const long long r = rb + lane;
    int len = 0, key = -1 - lane;            // lanes without a row get keys of their own
    if (r < r1) {
      len = __ldg(row_ptr + r + 1) - __ldg(row_ptr + r);
      const int kq = quad_key(len);
      if (kq >= 0) key = kq;
    }
    const unsigned peers = __match_any_sync(FULL, key);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    int base = 0;
    if (key >= 0) base = s_next[warp][key];
    __syncwarp();
    if (key >= 0 && rank == 0) s_next[warp][key] = base + __popc(peers);
    __syncwarp();
    if (key >= 0) {
      row_of[base + rank] = (int)r;
      len_of[base + rank] = len;
    }
  }
}

// quads[b] = quads of block b of `gpw` list slots: gpw times those of its first (longest) row; quads[blocks] = 0.
__global__ void __launch_bounds__(256) quad_order_block_quads_kernel(const int* __restrict__ len_of, int blocks, int gpw, int* __restrict__ quads) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b > blocks) return;
  quads[b] = b < blocks ? ((len_of[(long long)b * gpw] + 3) >> 2) * gpw : 0;
}

// Column-locality probe for matrices with short rows: for `samples` evenly spaced pairs of adjacent rows (r, r + 1),
// counts the entries of row r + 1 whose 128-byte line of x (32 four-byte entries) is also touched by row r.
// Banded / stencil / mesh matrices score near 1, matrices with random columns near 0.  out[0] += hits, out[1] += entries.
__global__ void __launch_bounds__(128) plan_col_locality_kernel(const int* __restrict__ row_ptr, const int* __restrict__ col_idx, int m,
                                                                int samples, unsigned long long* __restrict__ out) {
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= samples || m < 2) return;
  const long long r = (long long)s * (m - 1) / samples;
  const int a0 = row_ptr[r], a1 = row_ptr[r + 1], b1 = row_ptr[r + 2];
  const int la = a1 - a0, lb = b1 - a1;
  if (la <= 0 || lb <= 0 || la > 64 || lb > 64) return;
  unsigned hits = 0;
  for (int j = 0; j < lb; ++j) {
    const int line = col_idx[a1 + j] >> 5;
    bool found = false;
    for (int i = 0; i < la; ++i) found |= (col_idx[a0 + i] >> 5) == line;
    hits += found;
  }
  atomicAdd(&out[0], (unsigned long long)hits);
  atomicAdd(&out[1], (unsigned long long)lb);
}

// CSR content check on request.
__global__ void __launch_bounds__(256) validate_csr_kernel(const int* __restrict__ row_ptr, const int* __restrict__ col_idx, int m, int n,
                                                           int nnz, int* bad) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  int b = 0;
  if (i0 == 0) { if (row_ptr[0] != 0) b |= 1; if (row_ptr[m] != nnz) b |= 2; }
  for (long long i = i0; i < m; i += stride) if (row_ptr[i + 1] < row_ptr[i]) b |= 4;
  for (long long p = i0; p < nnz; p += stride) { const int c = col_idx[p]; if (c < 0 || c >= n) b |= 8; }
  if (b) atomicOr(bad, b);
}

}  // namespace b200sp
