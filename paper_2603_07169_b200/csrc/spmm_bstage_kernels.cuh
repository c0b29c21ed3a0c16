// SpMM with the slice of B held in shared memory (for matrices with few columns):
// Y = alpha * A * B + beta * Y  (paper, Appendix C, Table 6, task 13 -- its own shapes have 2048 columns
// and K = 4096 -- with alpha/beta).
//
// When A has few columns, a slice of LANES * 16 bytes of every row of B fits in one SM's shared memory
// (n * LANES * 16 bytes).  A CTA owns one such slice and one chunk of A's rows: a single thread fetches the
// slice with 2-D tiled bulk-tensor copies (TMA; box = slice width x 256 rows of B) behind an mbarrier, then
// groups of LANES lanes walk their rows of A and read B from shared memory (about an order of magnitude
// more gathers per clock than the L1-miss path), keeping VEC columns per lane in FP32 registers.  B is read
// from L2 / HBM once per (slice, row chunk) instead of once per nonzero.
//
// The (col, val) pairs of A go through shared memory too: a warp's 32 / LANES groups own consecutive rows,
// whose nonzeros are contiguous, so the warp first copies that range with coalesced loads into a buffer of
// its own (capw entries, carved from the shared memory the slice of B leaves) and the groups then read their
// pairs from there.  Read directly, the same pairs cost one L1 wavefront per group and request -- 40 % of the
// L1 data pipe this kernel is bound by.  No CTA-wide barrier is involved: warps stay independent.  A set of
// rows that does not fit the buffer (or capw = 0) is read from global memory as before.
#pragma once
#include <cuda.h>

#include "pipeline.cuh"
#include "spmm_kernels.cuh"

namespace b200sp {

__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap* map, int x, int y, unsigned bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}

template <typename T> struct RawFromSmem;
template <> struct RawFromSmem<float> { typedef float4 type; };
template <> struct RawFromSmem<bf16_t> { typedef uint4 type; };

// Dynamic shared memory: [ slice of B: bslice_bytes | per warp: (capw + 4) ints, (capw + 4) values ]; capw + 4 is a multiple of 8.
template <typename T, int VEC, int LANES, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmm_bstage_kernel(const __grid_constant__ CUtensorMap tmapB, int m, int n, int k, int row_chunks, int rows_per_chunk, int box_rows,
                   int bslice_bytes, int capw, const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                   const T* __restrict__ vals, T* __restrict__ Y, float alpha, float beta, int* __restrict__ err, int spin_limit,
                   int no_copies) {
  constexpr int KS = LANES * VEC, ROW_BYTES = LANES * 16, GPW = 32 / LANES, WARPS = THREADS / 32;
  constexpr unsigned FULL = 0xFFFFFFFFu;
  typedef typename RawVec<T, VEC>::type raw_t;
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long bar;
  const int tid = threadIdx.x;
  const int slice = blockIdx.x / row_chunks, chunk = blockIdx.x - slice * row_chunks;
  const int col_base = slice * KS;
  if (tid == 0) { mbar_init(smem_addr(&bar), 1); mbar_init_fence(); }
  __syncthreads();
  grid_dependency_wait();   // nothing above touches global memory
  if (tid == 0 && !no_copies) {   // no_copies (a test switch): nothing is issued, the wait below runs out with nothing in flight
    const int boxes = (n + box_rows - 1) / box_rows;
    mbar_arrive_expect_tx(smem_addr(&bar), (unsigned)boxes * (unsigned)box_rows * ROW_BYTES);   // rows past n are zero-filled and still counted
    for (int b = 0; b < boxes; ++b)
      tma_load_2d(smem_addr(smem + (size_t)b * box_rows * ROW_BYTES), &tmapB, col_base, b * box_rows, smem_addr(&bar));
  }
  const bool arrived = mbar_wait_bounded(smem_addr(&bar), 0, spin_limit);
  if (!__syncthreads_and(arrived)) {
    if (tid == 0) atomicExch(err, 1);
    (void)mbar_wait_bounded(smem_addr(&bar), 0, spin_limit);   // bounded second chance for the copies in flight
    return;
  }
  const int warp = tid >> 5, lane = tid & 31;
  const int gl = lane / LANES, l = lane % LANES;     // group inside the warp, lane inside the group
  const int col0 = col_base + l * VEC;
  const bool active = col0 < k;
  const unsigned char* Bs = smem + l * 16;
  const int entries = capw + 4;
  int* wcol = (int*)(smem + bslice_bytes + (size_t)warp * entries * (4 + sizeof(T)));
  T* wval = (T*)(wcol + entries);
  const int r_begin = chunk * rows_per_chunk;
  const int r_end = min(m, r_begin + rows_per_chunk);
  for (int rb = r_begin + warp * GPW; rb < r_end; rb += WARPS * GPW) {   // GPW consecutive rows per warp and step
    int bound = 0;
    if (lane <= GPW) bound = __ldg(row_ptr + min(rb + lane, r_end));     // rows past the chunk's end come out empty
    const int a = __shfl_sync(FULL, bound, 0), b_end = __shfl_sync(FULL, bound, GPW);
    const int rs = __shfl_sync(FULL, bound, gl), re = __shfl_sync(FULL, bound, gl + 1);
    const int row = rb + gl;
    float acc[VEC], tot[VEC];   // acc: the current block of at most kChainBlock products; tot: the sum of the completed blocks
#pragma unroll
    for (int j = 0; j < VEC; ++j) { acc[j] = 0.0f; tot[j] = 0.0f; }
    int fold = 0;
    if (capw > 0 && b_end - a <= capw) {
      // ---- the warp's nonzeros [a, b_end) into its buffer; entry p sits at p - (a & ~3), so p & 3 is kept
      const int a4 = a & ~3;
      __syncwarp();                      // the previous step's readers are done with the buffer
#pragma unroll 4
      for (int p = a + lane; p < b_end; p += 32) {
        wcol[p - a4] = __ldg(col_idx + p);
        wval[p - a4] = __ldg(vals + p);
      }
      __syncwarp();
      int q = rs - a4;
      const int qe = re - a4;
      for (; q < qe && (q & 3); ++q) {
        const raw_t b = *(const raw_t*)(Bs + (size_t)wcol[q] * ROW_BYTES);
        RawVec<T, VEC>::fma_mixed(b, to_f32(wval[q]), acc);
      }
      for (; q + 4 <= qe; q += 4) {
        if (++fold > kChainBlock / 4) {
          fold = 1;
#pragma unroll
          for (int j = 0; j < VEC; ++j) { tot[j] += acc[j]; acc[j] = 0.0f; }
        }
        int c[4]; float v[4];
        lds_a4(wcol, wval, q, c, v);   // (one pair per lane plus shuffles round the group was measured slower: 2.26 against 1.86 ms)
        raw_t b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) b[u] = *(const raw_t*)(Bs + (size_t)c[u] * ROW_BYTES);
#pragma unroll
        for (int u = 0; u < 4; ++u) RawVec<T, VEC>::fma_mixed(b[u], v[u], acc);
      }
      for (; q < qe; ++q) {
        const raw_t b = *(const raw_t*)(Bs + (size_t)wcol[q] * ROW_BYTES);
        RawVec<T, VEC>::fma_mixed(b, to_f32(wval[q]), acc);
      }
    } else {
      // ---- too many nonzeros for the buffer: pairs straight from global memory
      int p = rs;
      for (; p < re && (p & 3); ++p) {
        const raw_t b = *(const raw_t*)(Bs + (size_t)__ldg(col_idx + p) * ROW_BYTES);
        RawVec<T, VEC>::fma_mixed(b, to_f32(__ldg(vals + p)), acc);
      }
      for (; p + 4 <= re; p += 4) {
        if (++fold > kChainBlock / 4) {
          fold = 1;
#pragma unroll
          for (int j = 0; j < VEC; ++j) { tot[j] += acc[j]; acc[j] = 0.0f; }
        }
        int c[4]; float v[4];
        ld_a4(col_idx, vals, p, c, v);
        raw_t b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) b[u] = *(const raw_t*)(Bs + (size_t)c[u] * ROW_BYTES);
#pragma unroll
        for (int u = 0; u < 4; ++u) RawVec<T, VEC>::fma_mixed(b[u], v[u], acc);
      }
      for (; p < re; ++p) {
        const raw_t b = *(const raw_t*)(Bs + (size_t)__ldg(col_idx + p) * ROW_BYTES);
        RawVec<T, VEC>::fma_mixed(b, to_f32(__ldg(vals + p)), acc);
      }
    }
    if (active && row < r_end) {
      T* yp = Y + (long long)row * k + col0;
      float out[VEC];
#pragma unroll
      for (int j = 0; j < VEC; ++j) acc[j] += tot[j];
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
  }
}

}  // namespace b200sp
