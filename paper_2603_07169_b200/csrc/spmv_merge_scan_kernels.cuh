// Merge-tile CSR SpMV with an in-register segmented scan:
// y = alpha * A * x + beta * y  (paper, Appendix C, Table 6, task 12, with alpha/beta).
//
// Same tiles, split points, carries, tails and fix-up kernel as spmv_merge_tile_kernel; what differs is how
// the products of a tile are reduced by row.  Instead of parking every product in shared memory and adding
// them up row by row afterwards, the tile first marks the position of each row's last nonzero in a bitmap
// (one shared-memory atomic per non-empty row), then streams its nonzeros, gathers x and runs a segmented
// inclusive scan over the products: four per thread in registers, 32 lanes with __shfl_up, and the 128-wide
// chunks of the tile through a small shared array.  Only the scan value at each row end is written to shared
// memory, so the load/store pipe that the x gathers need is no longer shared with two accesses per nonzero.
// The order of additions is fixed by positions, so results are bit-reproducible.
#pragma once
#include "common.cuh"

namespace b200sp {

template <typename T, int ITEMS, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmv_merge_scan_kernel(int m, int nnz, const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                       const T* __restrict__ vals, const T* __restrict__ x, T* __restrict__ y, float alpha, float beta,
                       const int* __restrict__ split_row, float* __restrict__ carry, float* __restrict__ tail, int tile_stride) {
  constexpr int G = 4, U = 4, WARPS = THREADS / 32;
  constexpr int POS_N = ITEMS + 2 * G;              // local positions, counted from the aligned start a0
  constexpr int NCHUNK = (POS_N + 127) / 128 + 1;   // 128 positions per warp-wide chunk
  static_assert(NCHUNK <= 32, "the chunk scan is done by one warp");
  __shared__ float endval[POS_N];                   // scan value at each row-end position (other entries unused)
  __shared__ unsigned endbits[(POS_N + 31) / 32 + 1];
  __shared__ float chunk_tail[NCHUNK];              // sum after the chunk's last row end (the whole chunk if it has none)
  __shared__ int chunk_first[NCHUNK];               // position of the chunk's first row end, -1 if none

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // CTAs are dispatched in blockIdx order; walking the tiles with a stride coprime to their number mixes tiles from the
  // dense part of the matrix (gather-heavy) with tiles from the sparse part (row-heavy) on every SM at all times.
  const int t = (int)(((long long)blockIdx.x * tile_stride) % gridDim.x);
  const long long total = (long long)m + nnz;
  const long long d0 = (long long)t * ITEMS;
  const long long d1 = min(d0 + ITEMS, total);
  const int r0 = split_row[t], r1 = split_row[t + 1];
  const int p0 = (int)(d0 - r0), p1 = (int)(d1 - r1);
  const int a0 = p0 & ~(G - 1);

  for (int i = tid; i < (POS_N + 31) / 32 + 1; i += THREADS) endbits[i] = 0u;
  for (int i = tid; i < NCHUNK; i += THREADS) { chunk_tail[i] = 0.0f; chunk_first[i] = -1; }
  __syncthreads();

  // ---- mark the last nonzero of every non-empty row that ends in this tile and has products here
  for (int r = r0 + tid; r < r1; r += THREADS) {
    const int rs = __ldg(row_ptr + r), re = __ldg(row_ptr + r + 1);
    if (re > rs && re > p0) {
      const int pos = re - 1 - a0;
      atomicOr(&endbits[pos >> 5], 1u << (pos & 31));
    }
  }
  __syncthreads();

  // ---- products and segmented scan, one 128-position chunk per warp and step
  const int nq = (p1 - a0 + G - 1) / G;
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
    float pr[U][G];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int j = 0; j < G; ++j) pr[u][j] = ok[u][j] ? v[u][j] * ld_gather(x + c[u][j]) : 0.0f;

#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int q = qb + u * THREADS + tid;       // may be >= nq: then products and flags are zero, the lane only takes part in the shuffles
      const int lp = q * G;                        // local position of this lane's first product
      unsigned f = 0u;
      if (q < nq) f = (endbits[lp >> 5] >> (lp & 31)) & 0xFu;   // lp is a multiple of 4: the four bits sit in one word
      // the lane's own summary: sum after its last row end (all four if it has none)
      float tl = 0.0f;
#pragma unroll
      for (int j = 0; j < G; ++j) { tl += pr[u][j]; if (f & (1u << j)) tl = 0.0f; }
      // inclusive segmented scan over the lanes: (t1,e1) + (t2,e2) = (e2 ? t2 : t1 + t2, e1 | e2)
      float st = tl;
      unsigned se = f != 0u;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const float t2 = __shfl_up_sync(0xFFFFFFFFu, st, d);
        const unsigned e2 = __shfl_up_sync(0xFFFFFFFFu, se, d);
        if (lane >= d) { if (!se) st += t2; se |= e2; }
      }
      float cin = __shfl_up_sync(0xFFFFFFFFu, st, 1);   // carry into this lane from the lanes before it
      if (lane == 0) cin = 0.0f;
      // second pass over the four products: the value at each row end goes to shared memory
      float run = cin;
      int first_pos = -1;
#pragma unroll
      for (int j = 0; j < G; ++j) {
        run += pr[u][j];
        if (f & (1u << j)) { endval[lp + j] = run; if (first_pos < 0) first_pos = lp + j; run = 0.0f; }
      }
      // chunk summary: first row end of the chunk (it still lacks the carry from earlier chunks) and the open sum at its end
      const unsigned have = __ballot_sync(0xFFFFFFFFu, f != 0u);
      const int chunk = (qb + u * THREADS) / 32 + warp;
      if (have) {
        const int src = __ffs(have) - 1;
        const int fp = __shfl_sync(0xFFFFFFFFu, first_pos, src);
        if (lane == 0) chunk_first[chunk] = fp;          // a chunk with a row end always lies inside the tile: chunk < NCHUNK
      }
      if (lane == 31 && chunk < NCHUNK) chunk_tail[chunk] = st;
    }
  }
  __syncthreads();

  // ---- carries between the chunks of the tile (one warp), and the tile's own carry-out
  if (warp == 0) {
    const bool in = lane < NCHUNK;
    float st = in ? chunk_tail[lane] : 0.0f;
    const int fp = in ? chunk_first[lane] : -1;
    unsigned se = fp >= 0;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const float t2 = __shfl_up_sync(0xFFFFFFFFu, st, d);
      const unsigned e2 = __shfl_up_sync(0xFFFFFFFFu, se, d);
      if (lane >= d) { if (!se) st += t2; se |= e2; }
    }
    float cin = __shfl_up_sync(0xFFFFFFFFu, st, 1);
    if (lane == 0) cin = 0.0f;
    if (fp >= 0) endval[fp] += cin;                 // the chunk's first row end receives what the earlier chunks left open
    if (lane == NCHUNK - 1) carry[t] = r1 < m ? st : 0.0f;   // what is open at the end of the tile belongs to the unfinished row r1
  }
  __syncthreads();

  // ---- one thread per row: epilogue, or the tail of a row that began in an earlier tile
  for (int r = r0 + tid; r < r1; r += THREADS) {
    const int rs = __ldg(row_ptr + r), re = __ldg(row_ptr + r + 1);
    float acc = 0.0f;
    if (re > rs && re > p0) acc = endval[re - 1 - a0];
    if (rs < p0) tail[t] = acc;                      // completed by the fix-up kernel
    else epilogue_store(y, r, acc, alpha, beta);
  }
}

}  // namespace b200sp
