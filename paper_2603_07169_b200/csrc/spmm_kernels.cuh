// CSR SpMM kernel: Y = alpha * A * B + beta * Y, B (n x k) and Y (m x k) row-major
// (paper, Appendix C, Table 6, task 13, with alpha/beta).
//
// Lanes run along the dense dimension k: a group of LANES lanes owns one matrix row and each lane
// owns VEC consecutive columns of every CHUNK, so each read of a row of B and each write of a row
// of Y is one contiguous, vectorised, coalesced access.  Accumulators stay in FP32 registers.
#pragma once
#include "common.cuh"

namespace b200sp {

template <typename T, int VEC> struct VecLoad;
template <> struct VecLoad<float, 4> {
  static __device__ __forceinline__ void ld(const float* p, float (&v)[4]) { const float4 t = __ldg((const float4*)p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
  static __device__ __forceinline__ void ld_plain(const float* p, float (&v)[4]) { const float4 t = *(const float4*)p; v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
  static __device__ __forceinline__ void st(float* p, const float (&v)[4]) { *(float4*)p = make_float4(v[0], v[1], v[2], v[3]); }
};
template <> struct VecLoad<float, 1> {
  static __device__ __forceinline__ void ld(const float* p, float (&v)[1]) { v[0] = __ldg(p); }
  static __device__ __forceinline__ void ld_plain(const float* p, float (&v)[1]) { v[0] = *p; }
  static __device__ __forceinline__ void st(float* p, const float (&v)[1]) { *p = v[0]; }
};
template <> struct VecLoad<bf16_t, 8> {
  static __device__ __forceinline__ void unpack(const uint4 t, float (&v)[8]) {
    v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xFFFF0000u);
    v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xFFFF0000u);
    v[4] = __uint_as_float(t.z << 16); v[5] = __uint_as_float(t.z & 0xFFFF0000u);
    v[6] = __uint_as_float(t.w << 16); v[7] = __uint_as_float(t.w & 0xFFFF0000u);
  }
  static __device__ __forceinline__ void ld(const bf16_t* p, float (&v)[8]) { unpack(__ldg((const uint4*)p), v); }
  static __device__ __forceinline__ void ld_plain(const bf16_t* p, float (&v)[8]) { unpack(*(const uint4*)p, v); }
  static __device__ __forceinline__ unsigned pack2(float a, float b) {
    return (unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(a)) | ((unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(b)) << 16);
  }
  static __device__ __forceinline__ void st(bf16_t* p, const float (&v)[8]) {
    *(uint4*)p = make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
  }
};
template <> struct VecLoad<bf16_t, 1> {
  static __device__ __forceinline__ void ld(const bf16_t* p, float (&v)[1]) { v[0] = to_f32(__ldg(p)); }
  static __device__ __forceinline__ void ld_plain(const bf16_t* p, float (&v)[1]) { v[0] = to_f32(*p); }
  static __device__ __forceinline__ void st(bf16_t* p, const float (&v)[1]) { store_elem(p, v[0]); }
};

// No lane adds more than kChainBlock products in one sequential FP32 chain: longer rows are added block by block
// and the block sums are added in a second chain, so the worst-case rounding error of a row of L products is
// (kChainBlock + L / kChainBlock) * 2^-24 * sum|a b| instead of L * 2^-24 * sum|a b|.
constexpr int kChainBlock = 128;

// One group of LANES lanes per row; the group sweeps k in chunks of LANES * VEC columns, NCH chunks
// at a time held in registers (the row's nonzeros are re-read from L1 for each further block of chunks).
// Rows longer than long_thresh are left to spmm_long_row_kernel.
template <typename T, int VEC, int LANES, int NCH, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmm_row_group_kernel(int m, int k, const int* __restrict__ row_ptr, const int* __restrict__ col_idx, const T* __restrict__ vals,
                      const T* __restrict__ B, T* __restrict__ Y, float alpha, float beta, int long_thresh) {
  constexpr int GROUPS = THREADS / LANES;
  grid_dependency_wait();
  const int g = threadIdx.x / LANES, lane = threadIdx.x % LANES;
  const long long row = (long long)blockIdx.x * GROUPS + g;
  if (row >= m) return;
  const int rs = row_ptr[row], re = row_ptr[row + 1];
  if (re - rs > long_thresh) return;
  constexpr int SPAN = LANES * VEC;  // columns covered by one chunk
  for (int c0 = 0; c0 < k; c0 += SPAN * NCH) {
    float acc[NCH][VEC], tot[NCH][VEC];
#pragma unroll
    for (int h = 0; h < NCH; ++h)
#pragma unroll
      for (int j = 0; j < VEC; ++j) { acc[h][j] = 0.0f; tot[h][j] = 0.0f; }
    int p = rs;
    int fold = 0;
    for (; p + 4 <= re; p += 4) {  // four independent B rows in flight per lane
      if (++fold > kChainBlock / 4) {   // a block of products is complete: its sum joins the second-level chain
        fold = 1;
#pragma unroll
        for (int h = 0; h < NCH; ++h)
#pragma unroll
          for (int j = 0; j < VEC; ++j) { tot[h][j] += acc[h][j]; acc[h][j] = 0.0f; }
      }
      int cc[4]; float vv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { cc[u] = __ldg(col_idx + p + u); vv[u] = to_f32(__ldg(vals + p + u)); }
      float b[4][NCH][VEC];
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int h = 0; h < NCH; ++h) {
          const int col = c0 + h * SPAN + lane * VEC;
          if (col < k) VecLoad<T, VEC>::ld(B + (long long)cc[u] * k + col, b[u][h]);
          else {
#pragma unroll
            for (int j = 0; j < VEC; ++j) b[u][h][j] = 0.0f;
          }
        }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int h = 0; h < NCH; ++h)
#pragma unroll
          for (int j = 0; j < VEC; ++j) acc[h][j] = fmaf(vv[u], b[u][h][j], acc[h][j]);
    }
    for (; p < re; ++p) {
      const int cc = __ldg(col_idx + p);
      const float vv = to_f32(__ldg(vals + p));
#pragma unroll
      for (int h = 0; h < NCH; ++h) {
        const int col = c0 + h * SPAN + lane * VEC;
        if (col < k) {
          float b[VEC];
          VecLoad<T, VEC>::ld(B + (long long)cc * k + col, b);
#pragma unroll
          for (int j = 0; j < VEC; ++j) acc[h][j] = fmaf(vv, b[j], acc[h][j]);
        }
      }
    }
#pragma unroll
    for (int h = 0; h < NCH; ++h) {
      const int col = c0 + h * SPAN + lane * VEC;
      if (col < k) {
        float out[VEC];
        T* yp = Y + row * k + col;
#pragma unroll
        for (int j = 0; j < VEC; ++j) acc[h][j] += tot[h][j];
        if (beta != 0.0f) {
          float old[VEC];
          VecLoad<T, VEC>::ld_plain(yp, old);
#pragma unroll
          for (int j = 0; j < VEC; ++j) out[j] = alpha * acc[h][j] + beta * old[j];
        } else {
#pragma unroll
          for (int j = 0; j < VEC; ++j) out[j] = alpha * acc[h][j];
        }
        VecLoad<T, VEC>::st(yp, out);
      }
    }
  }
}

// Raw 16-byte pieces of a row of B, converted to FP32 only when they are consumed (keeps registers low).
template <typename T, int VEC> struct RawVec;
template <> struct RawVec<float, 4> {
  typedef float4 type;
  static __device__ __forceinline__ float4 ld(const float* p) { return __ldg((const float4*)p); }

  static __device__ __forceinline__ void fma(const float4& b, float v, float (&acc)[4]) {
    acc[0] = fmaf(v, b.x, acc[0]); acc[1] = fmaf(v, b.y, acc[1]); acc[2] = fmaf(v, b.z, acc[2]); acc[3] = fmaf(v, b.w, acc[3]);
  }
  static __device__ __forceinline__ void fma_mixed(const float4& b, float v, float (&acc)[4]) { fma(b, v, acc); }
};
template <> struct RawVec<bf16_t, 8> {
  typedef uint4 type;
  static __device__ __forceinline__ uint4 ld(const bf16_t* p) { return __ldg((const uint4*)p); }

  // acc += v * b for the two BF16 halves of one word with the mixed-precision FMA of sm_100 (BF16 factors, FP32
  // addend and result, one rounding): the same value as fmaf on the widened factors, without the widening.
  static __device__ __forceinline__ void fma2(unsigned short vb, unsigned w, float& a0, float& a1) {
    asm("{ .reg .b16 lo, hi;\n\t"
        "mov.b32 {lo, hi}, %3;\n\t"
        "fma.rn.f32.bf16 %0, %2, lo, %0;\n\t"
        "fma.rn.f32.bf16 %1, %2, hi, %1; }"
        : "+f"(a0), "+f"(a1) : "h"(vb), "r"(w));
  }
  static __device__ __forceinline__ void fma(const uint4& b, float v, float (&acc)[8]) {
    acc[0] = fmaf(v, __uint_as_float(b.x << 16), acc[0]); acc[1] = fmaf(v, __uint_as_float(b.x & 0xFFFF0000u), acc[1]);
    acc[2] = fmaf(v, __uint_as_float(b.y << 16), acc[2]); acc[3] = fmaf(v, __uint_as_float(b.y & 0xFFFF0000u), acc[3]);
    acc[4] = fmaf(v, __uint_as_float(b.z << 16), acc[4]); acc[5] = fmaf(v, __uint_as_float(b.z & 0xFFFF0000u), acc[5]);
    acc[6] = fmaf(v, __uint_as_float(b.w << 16), acc[6]); acc[7] = fmaf(v, __uint_as_float(b.w & 0xFFFF0000u), acc[7]);
  }
  // Same values through fma2.  Measured: 8 % faster in the kernel that keeps B in shared memory (which is not held to
  // 32 registers), 5-10 % slower in the register-capped k-sliced kernel, which therefore keeps fma().
  static __device__ __forceinline__ void fma_mixed(const uint4& b, float v, float (&acc)[8]) {
    const unsigned short vb = (unsigned short)(__float_as_uint(v) >> 16);   // v is a widened BF16 value: its upper half is the value itself
    fma2(vb, b.x, acc[0], acc[1]); fma2(vb, b.y, acc[2], acc[3]); fma2(vb, b.z, acc[4], acc[5]); fma2(vb, b.w, acc[6], acc[7]);
  }
};

// four consecutive (col, val) pairs with two broadcast vector loads (p a multiple of 4)
__device__ __forceinline__ void ld_a4(const int* col_idx, const float* vals, int p, int (&c)[4], float (&v)[4]) {
  const int4 cc = __ldg((const int4*)(col_idx + p));
  const float4 vv = __ldg((const float4*)(vals + p));
  c[0] = cc.x; c[1] = cc.y; c[2] = cc.z; c[3] = cc.w; v[0] = vv.x; v[1] = vv.y; v[2] = vv.z; v[3] = vv.w;
}
__device__ __forceinline__ void ld_a4(const int* col_idx, const bf16_t* vals, int p, int (&c)[4], float (&v)[4]) {
  const int4 cc = __ldg((const int4*)(col_idx + p));
  const uint2 vv = __ldg((const uint2*)(vals + p));
  c[0] = cc.x; c[1] = cc.y; c[2] = cc.z; c[3] = cc.w;
  v[0] = __uint_as_float(vv.x << 16); v[1] = __uint_as_float(vv.x & 0xFFFF0000u);
  v[2] = __uint_as_float(vv.y << 16); v[3] = __uint_as_float(vv.y & 0xFFFF0000u);
}

// k-sliced kernel.  The dense dimension is cut into slices of LANES * VEC columns: 128 bytes per row of B, one cache
// line, with the usual eight lanes per row; fewer lanes (4, 2, 1) when k itself is narrower than that, so that no lane idles.  blockIdx.x = slice * row_blocks + row block, so CTAs run slice by slice and the
// part of B that a slice touches (n lines) can stay in L2 while every row of A passes over it; the
// price is re-reading col_idx / vals once per slice.  Eight lanes own one row of A; all eight read the
// row's (col, val) pairs with the same 128-bit loads (a broadcast, served by L1), and each lane keeps its
// VEC columns of the slice in FP32 registers with four independent 16-byte reads of B in flight.
// Rows longer than long_thresh are left to spmm_long_row_kernel.
// acc += sum over nonzeros [p, pe) of vals[q] * (this lane's VEC columns of row col_idx[q] of B): scalar steps up to the
// first multiple of four, then four independent 16-byte reads of B in flight per lane.
template <typename T, int VEC>
__device__ __forceinline__ void slice_accumulate(const int* __restrict__ col_idx, const T* __restrict__ vals, const T* __restrict__ Bc, int k,
                                                 int p, int pe, float (&acc)[VEC]) {
  typedef typename RawVec<T, VEC>::type raw_t;
  for (; p < pe && (p & 3); ++p) {   // up to the first multiple of four
    const raw_t b = RawVec<T, VEC>::ld(Bc + (long long)__ldg(col_idx + p) * k);
    RawVec<T, VEC>::fma(b, to_f32(__ldg(vals + p)), acc);
  }
  for (; p + 4 <= pe; p += 4) {
    int c[4]; float v[4];
    ld_a4(col_idx, vals, p, c, v);
    raw_t b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) b[u] = RawVec<T, VEC>::ld(Bc + (long long)c[u] * k);
#pragma unroll
    for (int u = 0; u < 4; ++u) RawVec<T, VEC>::fma(b[u], v[u], acc);
  }
  for (; p < pe; ++p) {
    const raw_t b = RawVec<T, VEC>::ld(Bc + (long long)__ldg(col_idx + p) * k);
    RawVec<T, VEC>::fma(b, to_f32(__ldg(vals + p)), acc);
  }
}

template <typename T, int VEC>
__device__ __forceinline__ void slice_store(T* yp, const float (&acc)[VEC], float alpha, float beta) {
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

// four consecutive (col, val) pairs from a shared-memory buffer (index a multiple of 4)
__device__ __forceinline__ void lds_a4(const int* col_s, const float* val_s, int q, int (&c)[4], float (&v)[4]) {
  const int4 cc = *(const int4*)(col_s + q);
  const float4 vv = *(const float4*)(val_s + q);
  c[0] = cc.x; c[1] = cc.y; c[2] = cc.z; c[3] = cc.w; v[0] = vv.x; v[1] = vv.y; v[2] = vv.z; v[3] = vv.w;
}
__device__ __forceinline__ void lds_a4(const int* col_s, const bf16_t* val_s, int q, int (&c)[4], float (&v)[4]) {
  const int4 cc = *(const int4*)(col_s + q);
  const uint2 vv = *(const uint2*)(val_s + q);
  c[0] = cc.x; c[1] = cc.y; c[2] = cc.z; c[3] = cc.w;
  v[0] = __uint_as_float(vv.x << 16); v[1] = __uint_as_float(vv.x & 0xFFFF0000u);
  v[2] = __uint_as_float(vv.y << 16); v[3] = __uint_as_float(vv.y & 0xFFFF0000u);
}

// One vector of four consecutive stored values written to shared memory (q a multiple of 4).
__device__ __forceinline__ void sts_vals4(float* val_s, int q, const float* __restrict__ vals, int p) {
  *(float4*)(val_s + q) = __ldg((const float4*)(vals + p));
}
__device__ __forceinline__ void sts_vals4(bf16_t* val_s, int q, const bf16_t* __restrict__ vals, int p) {
  *(uint2*)(val_s + q) = __ldg((const uint2*)(vals + p));
}

// k-sliced kernel with the (col, val) pairs of A staged in shared memory.  In spmm_slice_kernel every step of a row's walk
// is two dependent memory latencies: the broadcast load of four (col, val) pairs, then the four reads of B they name -- and a
// row is a chain of such steps, which is what bounds that kernel (its reads of B never fill the L2-to-SM path).  Here a warp
// first copies the nonzeros of its 32 / LANES consecutive rows (they are contiguous in col_idx / vals) into a buffer of its own
// with coalesced 128-bit loads -- one latency for the whole set -- and the row walks then take their pairs from shared memory,
// so a step costs one latency, that of B.  Warps stay independent (no CTA-wide barrier).  A set of rows that does not fit the
// buffer (CAPW entries) is walked from global memory as in spmm_slice_kernel.  Measured on 2^19 rows of 32 nonzeros: BF16 5-6 %
// faster than spmm_slice_kernel, FP32 2-3 % slower (its buffers take more of L1), so it is the default for BF16 only.  Eight or
// sixteen reads of B in flight per lane at 48 / 80 registers were 3-30 % slower than four at 32: warps resident, not loads per
// warp, are what keeps the L2-to-SM path busy.
template <typename T, int VEC, int THREADS, int LANES, int CAPW>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS)
spmm_slice_staged_kernel(int m, int nnz, int k, int row_blocks, const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                         const T* __restrict__ vals, const T* __restrict__ B, T* __restrict__ Y, float alpha, float beta, int long_thresh) {
  constexpr int GROUPS = THREADS / LANES, KS = LANES * VEC, GPW = 32 / LANES, WARPS = THREADS / 32;
  constexpr unsigned FULL = 0xFFFFFFFFu;
  typedef typename RawVec<T, VEC>::type raw_t;
  __shared__ __align__(16) int col_s[WARPS][CAPW + 8];
  __shared__ __align__(16) T val_s[WARPS][CAPW + 8];
  grid_dependency_wait();
  const int slice = blockIdx.x / row_blocks, rb = blockIdx.x - slice * row_blocks;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gl = lane / LANES, l8 = lane % LANES;
  const long long row0 = (long long)rb * GROUPS + warp * GPW;        // first row of this warp
  if (row0 >= m) return;
  int bound = 0;
  if (lane <= GPW) bound = __ldg(row_ptr + min(row0 + lane, (long long)m));
  const int a = __shfl_sync(FULL, bound, 0), b_end = __shfl_sync(FULL, bound, GPW);
  const int rs = __shfl_sync(FULL, bound, gl), re = __shfl_sync(FULL, bound, gl + 1);
  const long long row = row0 + gl;
  const int col0 = slice * KS + l8 * VEC;
  const bool active = row < m && col0 < k && re - rs <= long_thresh;
  const T* Bc = B + col0;
  float acc[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
  const int a4 = a & ~3;
  if (b_end - a4 <= CAPW) {
    int* wcol = col_s[warp];
    T* wval = val_s[warp];
    const int nnz4 = nnz & ~3;
    for (int p = a4 + lane * 4; p < b_end; p += 128) {            // entry p sits at p - a4, so p & 3 is kept
      if (p + 4 <= nnz4) {
        *(int4*)(wcol + (p - a4)) = __ldg((const int4*)(col_idx + p));
        sts_vals4(wval, p - a4, vals, p);
      } else {
        for (int j = p; j < b_end; ++j) { wcol[j - a4] = __ldg(col_idx + j); wval[j - a4] = __ldg(vals + j); }
      }
    }
    __syncwarp();
    if (active) {
      int q = rs - a4;
      const int qe = re - a4;
      for (; q < qe && (q & 3); ++q) {
        const raw_t b = RawVec<T, VEC>::ld(Bc + (long long)wcol[q] * k);
        RawVec<T, VEC>::fma(b, to_f32(wval[q]), acc);
      }
      for (; q + 4 <= qe; q += 4) {
        int c[4]; float v[4];
        lds_a4(wcol, wval, q, c, v);
        raw_t b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) b[u] = RawVec<T, VEC>::ld(Bc + (long long)c[u] * k);
#pragma unroll
        for (int u = 0; u < 4; ++u) RawVec<T, VEC>::fma(b[u], v[u], acc);
      }
      for (; q < qe; ++q) {
        const raw_t b = RawVec<T, VEC>::ld(Bc + (long long)wcol[q] * k);
        RawVec<T, VEC>::fma(b, to_f32(wval[q]), acc);
      }
    }
  } else if (active) {
    slice_accumulate<T, VEC>(col_idx, vals, Bc, k, rs, re, acc);
  }
  if (active) slice_store<T, VEC>(Y + row * k + col0, acc, alpha, beta);
}

template <typename T, int VEC, int THREADS, int LANES>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS)
spmm_slice_kernel(int m, int k, int row_blocks, const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                  const T* __restrict__ vals, const T* __restrict__ B, T* __restrict__ Y, float alpha, float beta, int long_thresh) {
  constexpr int GROUPS = THREADS / LANES, KS = LANES * VEC;
  typedef typename RawVec<T, VEC>::type raw_t;
  grid_dependency_wait();
  const int slice = blockIdx.x / row_blocks, rb = blockIdx.x - slice * row_blocks;
  const int g = threadIdx.x / LANES, l8 = threadIdx.x % LANES;
  const long long row = (long long)rb * GROUPS + g;
  if (row >= m) return;
  const int rs = __ldg(row_ptr + row), re = __ldg(row_ptr + row + 1);
  if (re - rs > long_thresh) return;
  const int col0 = slice * KS + l8 * VEC;
  if (col0 >= k) return;
  const T* Bc = B + col0;
  float acc[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
  int p = rs;
  for (; p < re && (p & 3); ++p) {   // up to the first multiple of four
    const raw_t b = RawVec<T, VEC>::ld(Bc + (long long)__ldg(col_idx + p) * k);
    RawVec<T, VEC>::fma(b, to_f32(__ldg(vals + p)), acc);
  }
  for (; p + 4 <= re; p += 4) {
    int c[4]; float v[4];
    ld_a4(col_idx, vals, p, c, v);
    raw_t b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) b[u] = RawVec<T, VEC>::ld(Bc + (long long)c[u] * k);
#pragma unroll
    for (int u = 0; u < 4; ++u) RawVec<T, VEC>::fma(b[u], v[u], acc);
  }
  for (; p < re; ++p) {
    const raw_t b = RawVec<T, VEC>::ld(Bc + (long long)__ldg(col_idx + p) * k);
    RawVec<T, VEC>::fma(b, to_f32(__ldg(vals + p)), acc);
  }
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

// Column-range variant of the k-sliced kernel, for matrices whose rows hold their columns in ascending order.  When the
// part of B that one slice touches (n rows x 128 bytes) is larger than what L2 keeps, the columns are cut into `ranges`
// equal ranges and the kernel is launched once per range: launch r walks, in every row, only the nonzeros whose column lies
// in range r (row i: positions [cuts[(r-1) m + i], cuts[r m + i]), with the row's own bounds at both ends), so that all CTAs
// of a launch gather from the same n / ranges rows of B, which then stay in L2 while every row of A passes over them.
// Partial sums travel from launch to launch in FP32: in Y itself for FP32 storage (first range: Y = alpha acc + beta Y0,
// later ranges: Y += alpha acc), in `partial` (m x k floats) for BF16 storage, where Y is written once, by the last range,
// with a single rounding.  The launches are ordered by the stream; nothing inside one launch depends on another CTA.
template <typename T, int VEC, int THREADS, int LANES>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS)
spmm_slice_range_kernel(int m, int k, int row_blocks, int range, int ranges, const int* __restrict__ cuts,
                        const int* __restrict__ row_ptr, const int* __restrict__ col_idx, const T* __restrict__ vals,
                        const T* __restrict__ B, T* __restrict__ Y, float* __restrict__ partial, float alpha, float beta, int long_thresh) {
  constexpr int GROUPS = THREADS / LANES, KS = LANES * VEC;
  grid_dependency_wait();
  const int slice = blockIdx.x / row_blocks, rb = blockIdx.x - slice * row_blocks;
  const int g = threadIdx.x / LANES, l8 = threadIdx.x % LANES;
  const long long row = (long long)rb * GROUPS + g;
  if (row >= m) return;
  const int rs = __ldg(row_ptr + row), re = __ldg(row_ptr + row + 1);
  if (re - rs > long_thresh) return;
  const int col0 = slice * KS + l8 * VEC;
  if (col0 >= k) return;
  const int ps = range == 0 ? rs : __ldg(cuts + (long long)(range - 1) * m + row);
  const int pe = range == ranges - 1 ? re : __ldg(cuts + (long long)range * m + row);
  float acc[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
  slice_accumulate<T, VEC>(col_idx, vals, B + col0, k, ps, pe, acc);
  const long long o = row * k + col0;
  if constexpr (sizeof(T) == 4) {   // FP32 storage: Y carries the partial sums
    if (range == 0) {
      slice_store<T, VEC>(Y + o, acc, alpha, beta);
    } else {
      float old[VEC];
      VecLoad<T, VEC>::ld_plain(Y + o, old);
#pragma unroll
      for (int j = 0; j < VEC; ++j) old[j] = fmaf(alpha, acc[j], old[j]);
      VecLoad<T, VEC>::st(Y + o, old);
    }
  } else {                // BF16 storage: FP32 partial sums beside Y, one rounding at the end
    float* pp = partial + o;
    if (range > 0) {
#pragma unroll
      for (int j = 0; j < VEC; j += 4) {
        const float4 t = *reinterpret_cast<const float4*>(pp + j);
        acc[j] += t.x; acc[j + 1] += t.y; acc[j + 2] += t.z; acc[j + 3] += t.w;
      }
    }
    if (range == ranges - 1) {
      slice_store<T, VEC>(Y + o, acc, alpha, beta);
    } else {
#pragma unroll
      for (int j = 0; j < VEC; j += 4) *reinterpret_cast<float4*>(pp + j) = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
    }
  }
}

// Plan pass for the column ranges: for every row, the first position whose column is >= each range boundary
// (boundary j = ceil(j n / ranges), j = 1 .. ranges - 1; cuts[(j-1) m + row]), found by binary search, and a check that the
// row's columns ascend (ties allowed); *unsorted is raised otherwise, and the ranges are then not used.
__global__ void __launch_bounds__(256)
spmm_range_cuts_kernel(int m, int n, int ranges, const int* __restrict__ row_ptr, const int* __restrict__ col_idx, int* __restrict__ cuts,
                       int* __restrict__ unsorted) {
  const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= m) return;
  const int rs = row_ptr[row], re = row_ptr[row + 1];
  bool bad = false;
  for (int p = rs; p + 1 < re; ++p) bad |= col_idx[p] > col_idx[p + 1];
  if (bad) { atomicOr(unsorted, 1); return; }
  for (int j = 1; j < ranges; ++j) {
    const int bound = (int)(((long long)j * n + ranges - 1) / ranges);
    int lo = rs, hi = re;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (col_idx[mid] < bound) lo = mid + 1; else hi = mid; }
    cuts[(long long)(j - 1) * m + row] = lo;
  }
}

// The same lanes-along-k scheme for the rows of kChainBlock + 1 .. long-row threshold products, taken from the plan's list of
// such rows: the row is added in blocks of at most kChainBlock products (blocks end on multiples of four) and the block
// sums join a second-level chain.  A kernel of its own so that the second set of accumulators costs the register-capped
// kernel above nothing.
template <typename T, int VEC, int THREADS, int LANES>
__global__ void __launch_bounds__(THREADS)
spmm_medium_row_kernel(int num_rows, const int* __restrict__ rows, int k, int row_blocks, const int* __restrict__ row_ptr,
                       const int* __restrict__ col_idx, const T* __restrict__ vals, const T* __restrict__ B, T* __restrict__ Y,
                       float alpha, float beta) {
  constexpr int GROUPS = THREADS / LANES, KS = LANES * VEC;
  grid_dependency_wait();
  const int slice = blockIdx.x / row_blocks, rb = blockIdx.x - slice * row_blocks;
  const int g = threadIdx.x / LANES, l8 = threadIdx.x % LANES;
  const int idx = rb * GROUPS + g;
  if (idx >= num_rows) return;
  const long long row = rows[idx];
  const int rs = __ldg(row_ptr + row), re = __ldg(row_ptr + row + 1);
  const int col0 = slice * KS + l8 * VEC;
  if (col0 >= k) return;
  const T* Bc = B + col0;
  float acc[VEC], tot[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) { acc[j] = 0.0f; tot[j] = 0.0f; }
  for (int p = rs; p < re;) {
    const int pe = min(re, (p + kChainBlock) & ~3);
    slice_accumulate<T, VEC>(col_idx, vals, Bc, k, p, pe, acc);
#pragma unroll
    for (int j = 0; j < VEC; ++j) { tot[j] += acc[j]; acc[j] = 0.0f; }
    p = pe;
  }
  slice_store<T, VEC>(Y + row * k + col0, tot, alpha, beta);
}

// ---- nnz-balanced SpMM for irregular rows -------------------------------------------------------------------------------
// The k-sliced kernels above give every row to one group of eight lanes, so a row of a thousand nonzeros keeps its group busy
// long after its neighbours' rows of three are done, and empty rows idle the groups they were dealt.  Here the unit of work is
// a CHUNK of C consecutive nonzeros per lane group, whatever rows they belong to; a CTA owns a tile of GROUPS chunks.  A group
// walks its chunk row segment by row segment (the same vectorised inner loop), stores the rows that begin and end inside the
// chunk, and leaves two partial sums in shared memory: `head` for a first row that began before the chunk, `carry` for a last
// row that goes on after it.  After one barrier the group that holds a row's end adds the carries of the groups before it (in
// group order: reproducible) and stores the row; what crosses the tile's own ends goes to tile_tail / tile_carry in global
// memory and is finished by spmm_flat_fixup_kernel.  The rows are those that have nonzeros (m of them; row_ptr their m + 1
// offsets; row_id[r] the matrix row of list row r, or nullptr when every row of the matrix has nonzeros), so a tile holds at most
// TILE rows and all their bounds fit in shared memory; Y of the rows without nonzeros is written by spmm_empty_rows_kernel.
// No chain is longer than C products plus one term per group or tile that a row spans.
//   tile_row[t]  the list row that holds nonzero t * TILE, m for t * TILE >= nnz
template <typename T, int VEC, int THREADS, int C>
__global__ void __launch_bounds__(THREADS, 1536 / THREADS)
spmm_flat_kernel(int m, int nnz, int k, int tiles, const int* __restrict__ row_ptr, const int* __restrict__ row_id,
                 const int* __restrict__ tile_row, const int* __restrict__ col_idx, const T* __restrict__ vals, const T* __restrict__ B,
                 T* __restrict__ Y, float* __restrict__ tile_carry, float* __restrict__ tile_tail, float alpha, float beta) {
  constexpr int LANES = 8, GROUPS = THREADS / LANES, KS = LANES * VEC, TILE = GROUPS * C, RB = TILE + 32;
  __shared__ int rp_s[RB];                       // row_ptr[r_lo .. r_lo + RB): the bounds of the tile's rows (what does not fit is read from global memory)
  __shared__ float head_s[GROUPS][KS], carry_s[GROUPS][KS];
  __shared__ __align__(16) int col_s[TILE];      // the tile's (col, val) pairs, fetched once with coalesced 128-bit loads
  __shared__ __align__(16) T val_s[TILE];
  grid_dependency_wait();
  const int slice = blockIdx.x / tiles, t = blockIdx.x - slice * tiles;
  const int p_lo = t * TILE, p_hi = min(nnz, p_lo + TILE);
  const int r_lo = __ldg(tile_row + t);
  const int r_hi = min(__ldg(tile_row + t + 1), m - 1);
  {
    const int nnz4 = nnz & ~3;
    for (int i = threadIdx.x * 4; i < p_hi - p_lo; i += THREADS * 4) {
      const int p = p_lo + i;
      if (p + 4 <= nnz4) {
        *(int4*)(col_s + i) = ld_stream_i4(col_idx + p);
        sts_vals4(val_s, i, vals, p);
      } else {
        for (int u = 0; u < 4 && p + u < p_hi; ++u) { col_s[i + u] = __ldg(col_idx + p + u); val_s[i + u] = __ldg(vals + p + u); }
      }
    }
  }
  for (int j = threadIdx.x; j < RB && r_lo + j <= m; j += THREADS) rp_s[j] = __ldg(row_ptr + r_lo + j);
  __syncthreads();
  auto bound = [&](int r) { const int j = r - r_lo; return j < RB ? rp_s[j] : __ldg(row_ptr + r); };
  const int g = threadIdx.x / LANES, l8 = threadIdx.x % LANES;
  const int col0 = slice * KS + l8 * VEC;
  const bool active = col0 < k;
  const T* Bc = B + col0;
  const int c0 = p_lo + g * C, c1 = min(p_hi, c0 + C);
  typedef typename RawVec<T, VEC>::type raw_t;
  int head_row = -1, carry_rs = -1;              // the row whose end this chunk holds but whose start it does not; the start of the row it leaves unfinished
  bool has_carry = false;
  float acc[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
  if (c0 < c1) {
    int lo = r_lo, hi = r_hi;                    // the row that holds nonzero c0: the first r with row_ptr[r + 1] > c0
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (bound(mid + 1) <= c0) lo = mid + 1; else hi = mid; }
    int r = lo, rs = bound(r), re = bound(r + 1);
    // a row that has been added up to its last nonzero: stored if it began in this chunk, else left as the chunk's head
    auto finish_row = [&]() {
      if (rs >= c0) { if (active) slice_store<T, VEC>(Y + (long long)(row_id ? __ldg(row_id + r) : r) * k + col0, acc, alpha, beta); }
      else {
        head_row = r;
#pragma unroll
        for (int j = 0; j < VEC; ++j) head_s[g][l8 * VEC + j] = acc[j];
      }
#pragma unroll
      for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
    };
    // the chunk is walked four nonzeros at a time whatever rows they belong to (c0 is a multiple of four): the pairs come from
    // shared memory and four reads of B are in flight even where the rows are one or two nonzeros long
    for (int q = c0; q < c1; q += 4) {
      int c[4]; float v[4];
      lds_a4(col_s, val_s, q - p_lo, c, v);
      raw_t bv[4];
      if (active) {
#pragma unroll
        for (int u = 0; u < 4; ++u) bv[u] = RawVec<T, VEC>::ld(Bc + (long long)(q + u < c1 ? c[u] : c[0]) * k);   // past the chunk's end: any valid row of B
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int p = q + u;
        if (p < c1) {
          if (p == re) {                         // row r ended just before p: finish it and move to the row that holds p
            finish_row();
            do { ++r; rs = re; re = bound(r + 1); } while (re == rs);
          }
          if (active) RawVec<T, VEC>::fma(bv[u], v[u], acc);
        }
      }
    }
    if (re <= c1) finish_row();                  // the last row ends with the chunk
    else {                                       // or goes on after it
      has_carry = true;
      carry_rs = rs;
#pragma unroll
      for (int j = 0; j < VEC; ++j) carry_s[g][l8 * VEC + j] = acc[j];
    }
  }
  if (!has_carry) {
#pragma unroll
    for (int j = 0; j < VEC; ++j) carry_s[g][l8 * VEC + j] = 0.0f;
  }
  __syncthreads();
  const long long slot = ((long long)slice * tiles + t) * KS + l8 * VEC;
  if (head_row >= 0) {                           // complete the row that ends here: carries of the groups it passed through, in order, then the head
    const int rs = bound(head_row);
    const int j0 = rs >= p_lo ? (rs - p_lo) / C : 0;
#pragma unroll
    for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
    for (int u = j0; u < g; ++u) {
#pragma unroll
      for (int j = 0; j < VEC; ++j) acc[j] += carry_s[u][l8 * VEC + j];
    }
#pragma unroll
    for (int j = 0; j < VEC; ++j) acc[j] += head_s[g][l8 * VEC + j];
    if (rs >= p_lo) { if (active) slice_store<T, VEC>(Y + (long long)(row_id ? __ldg(row_id + head_row) : head_row) * k + col0, acc, alpha, beta); }
    else {
#pragma unroll
      for (int j = 0; j < VEC; ++j) tile_tail[slot + j] = acc[j];   // began in an earlier tile: finished by the fix-up kernel
    }
  }
  if (c0 < c1 && c1 == p_hi) {                   // the tile's last chunk: what the tile leaves unfinished
#pragma unroll
    for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
    if (has_carry) {
      const int j1 = carry_rs >= p_lo ? (carry_rs - p_lo) / C : 0;
      for (int u = j1; u <= g; ++u) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) acc[j] += carry_s[u][l8 * VEC + j];
      }
    }
#pragma unroll
    for (int j = 0; j < VEC; ++j) tile_carry[slot + j] = acc[j];
  }
}

// Finishes the rows that a tile boundary of spmm_flat_kernel cut: tile t holds the end of such a row when its first row began
// before the tile's first nonzero and ends inside the tile.  The row's value is tile_carry[first .. t-1] + tile_tail[t], the
// carries added in blocks of 16 whose sums form a second chain; one lane group per (slice, tile), fixed order.
template <typename T, int VEC, int THREADS, int TILE>
__global__ void __launch_bounds__(THREADS)
spmm_flat_fixup_kernel(int m, int nnz, int k, int tiles, int slices, const int* __restrict__ row_ptr, const int* __restrict__ row_id,
                       const int* __restrict__ tile_row, const float* __restrict__ tile_carry, const float* __restrict__ tile_tail,
                       T* __restrict__ Y, float alpha, float beta) {
  constexpr int LANES = 8, KS = LANES * VEC;
  grid_dependency_wait();
  const long long id = ((long long)blockIdx.x * THREADS + threadIdx.x) / LANES;
  const int l8 = threadIdx.x % LANES;
  if (id >= (long long)slices * tiles) return;
  const int slice = (int)(id / tiles), t = (int)(id - (long long)slice * tiles);
  if (t < 1) return;
  const int p_lo = t * TILE, p_hi = min(nnz, p_lo + TILE);
  const int r = tile_row[t];
  if (r >= m) return;
  const int rs = row_ptr[r], re = row_ptr[r + 1];
  if (rs >= p_lo || re > p_hi) return;           // the tile's first row begins inside it, or does not end in it
  const int col0 = slice * KS + l8 * VEC;
  if (col0 >= k) return;
  const int tf = rs / TILE;
  float acc[VEC], blk[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
  for (int u = tf; u < t; u += 16) {
#pragma unroll
    for (int j = 0; j < VEC; ++j) blk[j] = 0.0f;
    const int ue = min(u + 16, t);
    for (int v = u; v < ue; ++v) {
      const float* c = tile_carry + ((long long)slice * tiles + v) * KS + l8 * VEC;
#pragma unroll
      for (int j = 0; j < VEC; ++j) blk[j] += c[j];
    }
#pragma unroll
    for (int j = 0; j < VEC; ++j) acc[j] += blk[j];
  }
  const float* tl = tile_tail + ((long long)slice * tiles + t) * KS + l8 * VEC;
#pragma unroll
  for (int j = 0; j < VEC; ++j) acc[j] += tl[j];
  slice_store<T, VEC>(Y + (long long)(row_id ? row_id[r] : r) * k + col0, acc, alpha, beta);
}

// Y[i, :] = beta * Y[i, :] (zero when beta == 0) for the rows without nonzeros: the pass that goes with spmm_flat_kernel.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) spmm_empty_rows_kernel(int m, int k, const int* __restrict__ row_ptr, T* __restrict__ Y, float beta) {
  const int vecs = k / VEC;
  const long long total = (long long)m * vecs;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long row = i / vecs;
    if (__ldg(row_ptr + row) != __ldg(row_ptr + row + 1)) continue;
    float z[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) z[j] = 0.0f;
    slice_store<T, VEC>(Y + row * k + (i - row * vecs) * VEC, z, 0.0f, beta);
  }
}

// One CTA per (long row, slice): the CTA's groups of eight lanes stride over the row's nonzeros (sums in blocks of
// kChainBlock / 2 products, block sums in a second chain), then the per-group partial sums are combined pairwise through
// shared memory in a fixed tree (reproducible; five levels instead of a chain of 32).
template <typename T, int VEC, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmm_long_row_kernel(int k, int num_long, const int* __restrict__ long_rows, const int* __restrict__ row_ptr,
                     const int* __restrict__ col_idx, const T* __restrict__ vals, const T* __restrict__ B, T* __restrict__ Y,
                     float alpha, float beta) {
  constexpr int LANES = 8, GROUPS = THREADS / LANES, KS = LANES * VEC;
  __shared__ float part[GROUPS][KS];
  grid_dependency_wait();
  const int slice = blockIdx.x / num_long;
  const long long row = long_rows[blockIdx.x - slice * num_long];
  const int g = threadIdx.x / LANES, l8 = threadIdx.x % LANES;
  const int rs = __ldg(row_ptr + row), re = __ldg(row_ptr + row + 1);
  const int col0 = slice * KS + l8 * VEC;
  const bool active = col0 < k;
  const T* Bc = B + col0;
  float acc[VEC], tot[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) { acc[j] = 0.0f; tot[j] = 0.0f; }
  int fold = 0;
  for (int p = rs + g; p < re; p += GROUPS) {
    const int c = __ldg(col_idx + p);
    const float v = to_f32(__ldg(vals + p));
    if (++fold > kChainBlock / 2) {
      fold = 1;
#pragma unroll
      for (int j = 0; j < VEC; ++j) { tot[j] += acc[j]; acc[j] = 0.0f; }
    }
    if (active) {
      float b[VEC];
      VecLoad<T, VEC>::ld(Bc + (long long)c * k, b);
#pragma unroll
      for (int j = 0; j < VEC; ++j) acc[j] = fmaf(v, b[j], acc[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < VEC; ++j) part[g][l8 * VEC + j] = acc[j] + tot[j];
  __syncthreads();
  for (int half = GROUPS / 2; half > 0; half >>= 1) {
    for (int i = threadIdx.x; i < half * KS; i += THREADS) part[i / KS][i % KS] += part[i / KS + half][i % KS];
    __syncthreads();
  }
  if (threadIdx.x < KS) {
    const int col = slice * KS + threadIdx.x;
    if (col < k) epilogue_store(Y, row * k + col, part[0][threadIdx.x], alpha, beta);
  }
}

}  // namespace b200sp
