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

// One group of LANES lanes per row; the group sweeps k in chunks of LANES * VEC columns, NCH chunks
// at a time held in registers (the row's nonzeros are re-read from L1 for each further block of chunks).
template <typename T, int VEC, int LANES, int NCH, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmm_row_group_kernel(int m, int k, const int* __restrict__ row_ptr, const int* __restrict__ col_idx, const T* __restrict__ vals,
                      const T* __restrict__ B, T* __restrict__ Y, float alpha, float beta) {
  constexpr int GROUPS = THREADS / LANES;
  const int g = threadIdx.x / LANES, lane = threadIdx.x % LANES;
  const long long row = (long long)blockIdx.x * GROUPS + g;
  if (row >= m) return;
  const int rs = row_ptr[row], re = row_ptr[row + 1];
  constexpr int SPAN = LANES * VEC;  // columns covered by one chunk
  for (int c0 = 0; c0 < k; c0 += SPAN * NCH) {
    float acc[NCH][VEC];
#pragma unroll
    for (int h = 0; h < NCH; ++h)
#pragma unroll
      for (int j = 0; j < VEC; ++j) acc[h][j] = 0.0f;
    int p = rs;
    for (; p + 4 <= re; p += 4) {  // four independent B rows in flight per lane
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

}  // namespace b200sp
