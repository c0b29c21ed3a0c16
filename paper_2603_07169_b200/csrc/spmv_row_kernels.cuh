// Row-direct CSR SpMV kernel for matrices whose rows are all short (plan: max row length small):
// y = alpha * A * x + beta * y  (paper, Appendix C, Table 6, task 12, with alpha/beta).
//
// Persistent CTAs walk tiles of R consecutive rows.  For each tile one thread issues three bulk
// copies (TMA, 1-D) that bring the tile's row_ptr slice, col_idx range and vals range into a
// shared-memory stage; STAGES stages are in flight per CTA so the HBM stream never waits for the
// arithmetic.  Then one thread per row walks its nonzeros in shared memory, gathers x through the
// read-only path and accumulates in an FP32 register; consecutive lanes own consecutive rows, so
// for banded matrices a warp's gather touches one or two cache lines.  Rows never cross tiles, so
// there are no carries and no second kernel.  The summation order inside a row is fixed by the
// row's position, which keeps results bit-identical from run to run.
#pragma once
#include "pipeline.cuh"

namespace b200sp {

__host__ __device__ __forceinline__ int align16i(int b) { return (b + 15) & ~15; }

// Shared-memory bytes of one stage: row_ptr slice (R + 1 entries, padded), col_idx and vals ranges
// (cap entries: R * max_len plus slack for aligning the range to 8 entries at both ends).
template <typename T>
__host__ __device__ __forceinline__ int row_tile_stage_bytes(int R, int cap) {
  return align16i((R + 4) * 4) + align16i(cap * 4) + align16i(cap * (int)sizeof(T));
}

constexpr int kRowMaxStages = 4;

// One batch of UNROLL nonzeros of a row: shared-memory reads, then all gathers, then the FMA chain.
template <typename T, int UNROLL, bool ROT, bool FULL, bool ELL = false>
__device__ __forceinline__ float row_batch(const int* __restrict__ cp, const T* __restrict__ vp, const T* __restrict__ x,
                                           int j, int len, int rot, float acc) {
  int c[UNROLL];
  float v[UNROLL], xv[UNROLL];
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    const bool ok = FULL || (j + u < len);
    int q = j + u;
    if (ROT) { q += rot; if (q >= len) q -= len; }
    c[u] = ok ? cp[q] : -1;
    v[u] = ok ? to_f32(vp[q]) : 0.0f;
  }
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) xv[u] = ((FULL && !ELL) || c[u] >= 0) ? ld_gather(x + c[u]) : 0.0f;   // ELL: negative col_id = padding
  if (ELL) {
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) if (c[u] < 0) v[u] = 0.0f;   // a padded value may hold anything
  }
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) acc = fmaf(v[u], xv[u], acc);
  return acc;
}

// spin_limit bounds every barrier wait (polls); a wait that runs out sets *err and the CTA leaves.
// ELL = true: the matrix is ELL (row-major m x ell_width, padding col_id < 0): row i starts at i * ell_width,
// row_ptr is not read (the pointer may be null) and padded entries are skipped.
template <typename T, int THREADS, int UNROLL, bool ROT, bool ELL = false>
__global__ void __launch_bounds__(THREADS)
spmv_row_tile_kernel(int m, int nnz, const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                     const T* __restrict__ vals, const T* __restrict__ x, T* __restrict__ y, float alpha, float beta,
                     int R, int cap, int num_tiles, int stages, int rot_lanes, int* __restrict__ err, int ell_width, int spin_limit, int no_copies) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long full_bar[kRowMaxStages];
  const int tid = threadIdx.x;
  const int rp_bytes = align16i((R + 4) * 4), col_bytes = align16i(cap * 4);
  const int stage_bytes = row_tile_stage_bytes<T>(R, cap);
  const int my_tiles = (num_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int nnz8 = nnz & ~7;          // bulk copies stay inside [0, nnz8); the last < 8 entries go by plain loads
  const int rows4 = (m + 1) & ~3;     // same for row_ptr (m + 1 entries)

  if (tid == 0) {
    for (int s = 0; s < stages; ++s) mbar_init(smem_addr(&full_bar[s]), 1);
    mbar_init_fence();
  }
  __syncthreads();
  grid_dependency_wait();   // nothing above touches global memory

  // ---- producer (thread 0): stage i % stages <- tile blockIdx.x + i * gridDim.x
  int nb0 = 0, nb1 = 0;  // nonzero range of the next tile to issue (prefetched one step ahead)
  auto load_bounds = [&](int i) {
    if (i < my_tiles) {
      const int r0 = ((int)blockIdx.x + i * (int)gridDim.x) * R;
      if (ELL) { nb0 = r0 * ell_width; nb1 = min(r0 + R, m) * ell_width; }
      else { nb0 = __ldg(row_ptr + r0); nb1 = __ldg(row_ptr + min(r0 + R, m)); }
    }
  };
  auto issue = [&](int i, int s) {
    unsigned char* st = smem + (size_t)s * stage_bytes;
    int* rp_s = (int*)st;
    int* col_s = (int*)(st + rp_bytes);
    T* val_s = (T*)(st + rp_bytes + col_bytes);
    const unsigned bar = smem_addr(&full_bar[s]);
    const int r0 = ((int)blockIdx.x + i * (int)gridDim.x) * R;
    const int r1 = min(r0 + R, m);
    const int p0 = nb0, p1 = nb1;
    // row_ptr entries r0 .. r1 (inclusive)
    const int want = ELL ? 0 : r1 - r0 + 1;
    const int bulk_rows = ELL ? 0 : min((want + 3) & ~3, rows4 - r0);   // r0 is a multiple of 4
    for (int j = max(bulk_rows, 0); j < want; ++j) rp_s[j] = __ldg(row_ptr + r0 + j);
    // nonzeros [a0, a1) with a0, a1 multiples of 8 around [p0, p1)
    const int a0 = p0 & ~7;
    const int a1 = min((p1 + 7) & ~7, nnz8);
    const int bulk_nz = max(a1 - a0, 0);
    for (int p = max(a1, a0); p < p1; ++p) { col_s[p - a0] = __ldg(col_idx + p); val_s[p - a0] = __ldg(vals + p); }
    const unsigned bytes = (unsigned)(max(bulk_rows, 0) * 4 + bulk_nz * (4 + (int)sizeof(T)));
    fence_proxy_async_smem();
    mbar_arrive_expect_tx(bar, bytes);   // release: the plain stores above are visible to whoever observes the flip
    if (bulk_rows > 0) bulk_copy_g2s(smem_addr(rp_s), row_ptr + r0, (unsigned)bulk_rows * 4, bar);
    if (bulk_nz > 0) {
      bulk_copy_g2s(smem_addr(col_s), col_idx + a0, (unsigned)bulk_nz * 4, bar);
      bulk_copy_g2s(smem_addr(val_s), vals + a0, (unsigned)bulk_nz * (unsigned)sizeof(T), bar);
    }
  };
  // no_copies (a test switch): the producer issues nothing at all, so no copy can be in flight when the waits below run out
  if (tid == 0 && !no_copies) {
    load_bounds(0);
    for (int i = 0; i < stages && i < my_tiles; ++i) { issue(i, i); load_bounds(i + 1); }
  }

  const int lane = tid & 31;
  const int rot0 = (ROT && rot_lanes > 0) ? lane / rot_lanes : 0;   // cyclic start offset: spreads equal-length rows over the banks

  int s = 0;
  unsigned parity = 0;
  for (int i = 0; i < my_tiles; ++i) {
    unsigned char* st = smem + (size_t)s * stage_bytes;
    const int* rp_s = (const int*)st;
    const int* col_s = (const int*)(st + rp_bytes);
    const T* val_s = (const T*)(st + rp_bytes + col_bytes);
    const int r0 = ((int)blockIdx.x + i * (int)gridDim.x) * R;
    const int rows = min(R, m - r0);
    // y0 does not depend on the stage: fetch it before waiting
    float yold = 0.0f;
    if (beta != 0.0f && tid < rows) yold = to_f32(y[r0 + tid]);
    const bool arrived = mbar_wait_bounded(smem_addr(&full_bar[s]), parity, spin_limit);
    if (!__syncthreads_and(arrived)) {   // uniform decision: a wait ran out of polls
      if (tid == 0) atomicExch(err, 1);
      // give the copies already issued a bounded chance to land before the CTA (and its shared memory) goes away
      int s2 = s; unsigned par2 = parity;
      for (int k = 1; k < stages && i + k < my_tiles; ++k) {
        if (++s2 == stages) { s2 = 0; par2 ^= 1; }
        (void)mbar_wait_bounded(smem_addr(&full_bar[s2]), par2, spin_limit);
      }
      return;
    }
    if (tid < rows) {
      const int a0 = (ELL ? r0 * ell_width : rp_s[0]) & ~7;
      const int sft = (ELL ? (r0 + tid) * ell_width : rp_s[tid]) - a0;
      const int len = ELL ? ell_width : rp_s[tid + 1] - a0 - sft;
      const int* cp = col_s + sft;
      const T* vp = val_s + sft;
      const int rot = (ROT && rot0 < len) ? rot0 : 0;
      float acc = 0.0f;
      int j = 0;
      for (; j + UNROLL <= len; j += UNROLL) acc = row_batch<T, UNROLL, ROT, true, ELL>(cp, vp, x, j, len, rot, acc);
      if (j < len) acc = row_batch<T, UNROLL, ROT, false, ELL>(cp, vp, x, j, len, rot, acc);
      float r = alpha * acc;
      if (beta != 0.0f) r += beta * yold;
      store_elem(y + r0 + tid, r);
    }
    __syncthreads();   // every thread is done with stage s
    if (tid == 0 && !no_copies && i + stages < my_tiles) { issue(i + stages, s); load_bounds(i + stages + 1); }
    if (++s == stages) { s = 0; parity ^= 1; }
  }
}

}  // namespace b200sp
