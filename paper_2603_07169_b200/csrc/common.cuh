// Shared device helpers for the b200sp kernels: streaming / read-only loads and BF16 storage access.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace b200sp {

typedef unsigned short bf16_t;  // raw bfloat16 bit pattern

// ---- element traits: storage type -> FP32 and back (one round-to-nearest-even at the store) ----
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16_t v) { return __uint_as_float(((unsigned)v) << 16); }
__device__ __forceinline__ void store_elem(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_elem(bf16_t* p, float v) { *p = __bfloat16_as_ushort(__float2bfloat16_rn(v)); }

// ---- streaming loads: read once, keep out of L1 so that L1 holds the gathered operand ----
__device__ __forceinline__ int4 ld_stream_i4(const int* p) {
  int4 v;
  asm("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ int ld_stream_i1(const int* p) {
  int v;
  asm("ld.global.nc.L1::no_allocate.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
// four consecutive stored values -> four floats
__device__ __forceinline__ void ld_stream_vals4(const float* p, float (&v)[4]) {
  asm("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]) : "l"(p));
}
__device__ __forceinline__ void ld_stream_vals4(const bf16_t* p, float (&v)[4]) {
  unsigned a, b;
  asm("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(a), "=r"(b) : "l"(p));
  v[0] = __uint_as_float(a << 16); v[1] = __uint_as_float(a & 0xFFFF0000u);
  v[2] = __uint_as_float(b << 16); v[3] = __uint_as_float(b & 0xFFFF0000u);
}
__device__ __forceinline__ float ld_stream_val1(const float* p) {
  float v;
  asm("ld.global.nc.L1::no_allocate.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ float ld_stream_val1(const bf16_t* p) {
  unsigned short v;
  asm("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(v) : "l"(p));
  return __uint_as_float(((unsigned)v) << 16);
}

// ---- gathered operand (x, rows of B): read-only path, allocate in L1 ----
__device__ __forceinline__ float ld_gather(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ld_gather(const bf16_t* p) { return __uint_as_float(((unsigned)__ldg(p)) << 16); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// For kernels launched with programmatic stream serialisation: wait until every earlier kernel of the stream has
// completed and its writes are visible, then allow the next such kernel to be scheduled behind this one.  Without
// that launch attribute both instructions do nothing.
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
}

// y = alpha * acc + beta * y0 with the BLAS rule that beta == 0 never reads y0.
template <typename T>
__device__ __forceinline__ void epilogue_store(T* y, long long i, float acc, float alpha, float beta) {
  float r = alpha * acc;
  if (beta != 0.0f) r += beta * to_f32(y[i]);
  store_elem(y + i, r);
}

}  // namespace b200sp
