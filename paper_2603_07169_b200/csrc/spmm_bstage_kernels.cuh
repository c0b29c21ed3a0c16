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

template <typename T, int VEC, int LANES, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmm_bstage_kernel(const __grid_constant__ CUtensorMap tmapB, int m, int n, int k, int row_chunks, int rows_per_chunk, int box_rows,
                   const int* __restrict__ row_ptr, const int* __restrict__ col_idx, const T* __restrict__ vals, T* __restrict__ Y,
                   float alpha, float beta, int* __restrict__ err) {
  constexpr int GROUPS = THREADS / LANES, KS = LANES * VEC, ROW_BYTES = LANES * 16;
  typedef typename RawVec<T, VEC>::type raw_t;
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long bar;
  const int tid = threadIdx.x;
  const int slice = blockIdx.x / row_chunks, chunk = blockIdx.x - slice * row_chunks;
  const int col_base = slice * KS;
  if (tid == 0) { mbar_init(smem_addr(&bar), 1); mbar_init_fence(); }
  __syncthreads();
  if (tid == 0) {
    const int boxes = (n + box_rows - 1) / box_rows;
    mbar_arrive_expect_tx(smem_addr(&bar), (unsigned)boxes * (unsigned)box_rows * ROW_BYTES);   // rows past n are zero-filled and still counted
    for (int b = 0; b < boxes; ++b)
      tma_load_2d(smem_addr(smem + (size_t)b * box_rows * ROW_BYTES), &tmapB, col_base, b * box_rows, smem_addr(&bar));
  }
  const bool arrived = mbar_wait_bounded(smem_addr(&bar), 0);
  if (!__syncthreads_and(arrived)) {
    if (tid == 0) atomicExch(err, 1);
    (void)mbar_wait_bounded(smem_addr(&bar), 0);   // bounded second chance for the copies in flight
    return;
  }
  const int g = tid / LANES, l = tid % LANES;
  const int col0 = col_base + l * VEC;
  const bool active = col0 < k;
  const unsigned char* Bs = smem + l * 16;
  const int r_begin = chunk * rows_per_chunk;
  const int r_end = min(m, r_begin + rows_per_chunk);
  for (int row = r_begin + g; row < r_end; row += GROUPS) {
    const int rs = __ldg(row_ptr + row), re = __ldg(row_ptr + row + 1);
    float acc[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
    int p = rs;
    for (; p < re && (p & 3); ++p) {
      const raw_t b = *(const raw_t*)(Bs + (size_t)__ldg(col_idx + p) * ROW_BYTES);
      RawVec<T, VEC>::fma(b, to_f32(__ldg(vals + p)), acc);
    }
    for (; p + 4 <= re; p += 4) {
      int c[4]; float v[4];
      ld_a4(col_idx, vals, p, c, v);
      raw_t b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) b[u] = *(const raw_t*)(Bs + (size_t)c[u] * ROW_BYTES);
#pragma unroll
      for (int u = 0; u < 4; ++u) RawVec<T, VEC>::fma(b[u], v[u], acc);
    }
    for (; p < re; ++p) {
      const raw_t b = *(const raw_t*)(Bs + (size_t)__ldg(col_idx + p) * ROW_BYTES);
      RawVec<T, VEC>::fma(b, to_f32(__ldg(vals + p)), acc);
    }
    if (active) {
      T* yp = Y + (long long)row * k + col0;
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
  }
}

}  // namespace b200sp
