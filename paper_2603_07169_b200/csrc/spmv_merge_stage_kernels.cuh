// Persistent, staged merge-tile CSR SpMV kernel for matrices with long or very uneven rows:
// y = alpha * A * x + beta * y  (paper, Appendix C, Table 6, task 12, with alpha/beta).
//
// Same decomposition as spmv_merge_tile_kernel (tiles of ITEMS merge items over row ends + nonzeros,
// split points from the plan, carries / tails completed by spmv_carry_fixup_kernel), but each CTA is
// persistent and walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...: one thread issues 1-D bulk
// copies (TMA) of the tile's col_idx and vals ranges into a ring of shared-memory stages, so the HBM
// stream runs ahead of the arithmetic and the gather pipe is not idle while a tile's indices arrive.
//   phase 1  every thread takes groups of four staged nonzeros (128-bit shared loads), gathers x
//            through the read-only path and writes the products over the staged indices;
//   phase 2  one thread per row whose end lies in the tile adds short rows sequentially (the row's
//            bounds were fetched from row_ptr before phase 1, so their latency is hidden);
//   phase 3  one warp per long segment (lane-strided sums + __shfl_xor), then the unfinished row at
//            the tile's end goes to carry[t].
// All waits on the copy barriers are bounded; on a timeout the CTA records it in *err and leaves.
#pragma once
#include "pipeline.cuh"

namespace b200sp {

constexpr int kMergeMaxStages = 4;

template <typename T>
__host__ __device__ __forceinline__ int merge_stage_bytes(int items) {
  return (items + 16) * 4 + (((items + 16) * (int)sizeof(T) + 15) & ~15);
}

__device__ __forceinline__ void lds_vals4(const float* p, float (&v)[4]) { const float4 t = *(const float4*)p; v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
__device__ __forceinline__ void lds_vals4(const bf16_t* p, float (&v)[4]) {
  const uint2 t = *(const uint2*)p;
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xFFFF0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xFFFF0000u);
}

template <typename T, int ITEMS, int THREADS, int SHORT_MAX>
__global__ void __launch_bounds__(THREADS)
spmv_merge_stage_kernel(int m, int nnz, const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                        const T* __restrict__ vals, const T* __restrict__ x, T* __restrict__ y, float alpha, float beta,
                        const int* __restrict__ split_row, float* __restrict__ carry, float* __restrict__ tail,
                        int num_tiles, int stages, int* __restrict__ err) {
  constexpr int CAP = ITEMS + 16;
  constexpr int MAX_LONG = ITEMS / (SHORT_MAX + 1) + 2;
  constexpr int WARPS = THREADS / 32;
  constexpr int U = 2;
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long full_bar[kMergeMaxStages];
  __shared__ int long_rows[MAX_LONG];      // row index of each long segment
  __shared__ int2 long_span[MAX_LONG];     // its products: local [first, last) ; first < 0 marks "row began in an earlier tile"
  __shared__ int n_long;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int stage_bytes = merge_stage_bytes<T>(ITEMS);
  const int my_tiles = (num_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const long long total = (long long)m + nnz;
  const int nnz8 = nnz & ~7;

  if (tid == 0) {
    for (int s = 0; s < stages; ++s) mbar_init(smem_addr(&full_bar[s]), 1);
    mbar_init_fence();
    n_long = 0;
  }
  __syncthreads();

  auto tile_of = [&](int i) { return (int)blockIdx.x + i * (int)gridDim.x; };

  // ---- producer (thread 0): its own look-ahead on the split points
  int pb0 = 0, pb1 = 0;
  auto producer_bounds = [&](int i) {
    if (i < my_tiles) { const int t = tile_of(i); pb0 = __ldg(split_row + t); pb1 = __ldg(split_row + t + 1); }
  };
  auto issue = [&](int i, int s) {
    const int t = tile_of(i);
    const long long d0 = (long long)t * ITEMS;
    const long long d1 = min(d0 + ITEMS, total);
    const int p0 = (int)(d0 - pb0), p1 = (int)(d1 - pb1);
    unsigned char* st = smem + (size_t)s * stage_bytes;
    int* col_s = (int*)st;
    T* val_s = (T*)(st + CAP * 4);
    const unsigned bar = smem_addr(&full_bar[s]);
    const int a0 = p0 & ~7;
    const int a1 = min((p1 + 7) & ~7, nnz8);
    const int bulk = max(a1 - a0, 0);
    for (int p = max(a1, a0); p < p1; ++p) { col_s[p - a0] = __ldg(col_idx + p); val_s[p - a0] = __ldg(vals + p); }
    fence_proxy_async_smem();
    mbar_arrive_expect_tx(bar, (unsigned)(bulk * (4 + (int)sizeof(T))));
    if (bulk > 0) {
      bulk_copy_g2s(smem_addr(col_s), col_idx + a0, (unsigned)bulk * 4, bar);
      bulk_copy_g2s(smem_addr(val_s), vals + a0, (unsigned)bulk * (unsigned)sizeof(T), bar);
    }
  };
  if (tid == 0) {
    producer_bounds(0);
    for (int i = 0; i < stages && i < my_tiles; ++i) { issue(i, i); producer_bounds(i + 1); }
  }

  // ---- consumers: split points one tile ahead
  int nr0 = __ldg(split_row + tile_of(0)), nr1 = __ldg(split_row + tile_of(0) + 1);
  int s = 0;
  unsigned parity = 0;
  for (int i = 0; i < my_tiles; ++i) {
    const int t = tile_of(i);
    const int r0 = nr0, r1 = nr1;
    if (i + 1 < my_tiles) { nr0 = __ldg(split_row + tile_of(i + 1)); nr1 = __ldg(split_row + tile_of(i + 1) + 1); }
    const long long d0 = (long long)t * ITEMS;
    const long long d1 = min(d0 + ITEMS, total);
    const int p0 = (int)(d0 - r0), p1 = (int)(d1 - r1);
    const int a0 = p0 & ~7;
    // row bounds for phase 2 and the start of the unfinished row for phase 3, fetched now so that their
    // latency hides behind the copy wait and phase 1: thread tid owns rows r0 + tid + k * THREADS
    constexpr int KMAX = ITEMS / THREADS;
    int rsk[KMAX], re_last[KMAX];
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      const int r = r0 + tid + k * THREADS;
      rsk[k] = r <= r1 && r <= m ? __ldg(row_ptr + r) : 0;                       // r == r1 included: it is the neighbour's row end
      re_last[k] = (lane == 31 && r < r1) ? __ldg(row_ptr + r + 1) : 0;
    }
    const int carry_start = r1 < m ? __ldg(row_ptr + r1) : 0;

    unsigned char* st = smem + (size_t)s * stage_bytes;
    int* col_s = (int*)st;
    const T* val_s = (const T*)(st + CAP * 4);
    float* prod = (float*)col_s;   // products overwrite the staged indices

    const bool arrived = mbar_wait_bounded(smem_addr(&full_bar[s]), parity);
    if (!__syncthreads_and(arrived)) {
      if (tid == 0) atomicExch(err, 1);
      int s2 = s; unsigned par2 = parity;
      for (int k = 1; k < stages && i + k < my_tiles; ++k) {
        if (++s2 == stages) { s2 = 0; par2 ^= 1; }
        (void)mbar_wait_bounded(smem_addr(&full_bar[s2]), par2);
      }
      return;
    }
    // every thread has left the previous tile: its stage can be refilled, and the long-row list reset
    if (tid == 0) {
      n_long = 0;
      if (i > 0 && i - 1 + stages < my_tiles) {
        issue(i - 1 + stages, s == 0 ? stages - 1 : s - 1);
        producer_bounds(i + stages);
      }
    }

    // ---- phase 1
    const int lim = p1 - a0;
    const int nq = (lim + 3) >> 2;
    for (int qb = 0; qb < nq; qb += THREADS * U) {
      int4 c[U];
      float v[U][4], xv[U][4];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int q = qb + u * THREADS + tid;
        if (q < nq) { c[u] = *(const int4*)(col_s + 4 * q); lds_vals4(val_s + 4 * q, v[u]); }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int q = qb + u * THREADS + tid;
        if (q < nq) {
          if (4 * q + 4 <= lim) {
            xv[u][0] = ld_gather(x + c[u].x); xv[u][1] = ld_gather(x + c[u].y);
            xv[u][2] = ld_gather(x + c[u].z); xv[u][3] = ld_gather(x + c[u].w);
          } else {   // last group of the tile: entries at or beyond lim were not staged
            xv[u][0] = 4 * q + 0 < lim ? ld_gather(x + c[u].x) : 0.0f;
            xv[u][1] = 4 * q + 1 < lim ? ld_gather(x + c[u].y) : 0.0f;
            xv[u][2] = 4 * q + 2 < lim ? ld_gather(x + c[u].z) : 0.0f;
            xv[u][3] = 0.0f;
          }
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int q = qb + u * THREADS + tid;
        if (q < nq) *(float4*)(prod + 4 * q) = make_float4(v[u][0] * xv[u][0], v[u][1] * xv[u][1], v[u][2] * xv[u][2], v[u][3] * xv[u][3]);
      }
    }
    __syncthreads();

    // ---- phase 2
    {
      const int kmax = (r1 - r0 + THREADS - 1) / THREADS;   // uniform over the CTA
#pragma unroll
      for (int k = 0; k < KMAX; ++k) {
        if (k < kmax) {
          const int r = r0 + tid + k * THREADS;
          const int rs = rsk[k];
          int re = __shfl_down_sync(0xFFFFFFFFu, rs, 1);   // the next lane's row start is this row's end
          if (lane == 31) re = re_last[k];
          if (r < r1) {
            const int sft = max(rs, p0);
            const int len = re - sft;
            if (len <= SHORT_MAX) {
              float acc = 0.0f;
              const float* pp = prod + (sft - a0);
              for (int j = 0; j < len; ++j) acc += pp[j];
              if (rs < p0) tail[t] = acc;
              else epilogue_store(y, r, acc, alpha, beta);
            } else {
              const int slot = atomicAdd(&n_long, 1);   // order of the list does not affect any value
              long_rows[slot] = rs < p0 ? -r - 1 : r;
              long_span[slot] = make_int2(sft - a0, re - a0);
            }
          }
        }
      }
    }
    __syncthreads();

    // ---- phase 3
    const int nl = n_long;
    for (int li = warp; li < nl; li += WARPS) {
      const int r = long_rows[li];
      const int2 span = long_span[li];
      float acc = 0.0f;
      for (int q = span.x + lane; q < span.y; q += 32) acc += prod[q];
      acc = warp_sum(acc);
      if (lane == 0) {
        if (r < 0) tail[t] = acc;                    // row began in an earlier tile
        else epilogue_store(y, r, acc, alpha, beta);
      }
    }
    if (warp == WARPS - 1) {
      float acc = 0.0f;
      if (r1 < m) {
        const int sft = max(carry_start, p0);
        for (int q = sft - a0 + lane; q < p1 - a0; q += 32) acc += prod[q];
        acc = warp_sum(acc);
      }
      if (lane == 0) carry[t] = acc;
    }
    if (++s == stages) { s = 0; parity ^= 1; }
  }
}

}  // namespace b200sp
