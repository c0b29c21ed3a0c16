// Measurement probes: the hardware rates that bound the SpMV / SpMM kernels, measured by kernels that do nothing else.
// They have no counterpart in the paper's operations; the paper's Appendix A sorts kernels by which rate limits them
// (compute, memory latency, memory bandwidth), and these probes give the denominators for this part.
//   probe_gather_kernel   random reads of a table: the rate at which an SM takes L1 misses (table >> L1), L1 hits (table fits L1)
//                         or shared-memory reads (table staged in shared memory) -- the bound on gathering x
//   probe_stream_kernel   coalesced 128-bit reads of a buffer: what a pure stream of the CSR arrays can reach at a given size
//   probe_spmv_gather_kernel  the gather phase of a CSR SpMV on the caller's arrays and nothing else (no row sums, no y)
//   probe_lines_kernel    random reads of whole 128-byte lines (or two / four consecutive ones) by groups of 8 (16 / 32) lanes: the L2-to-SM path
//                         that SpMM's reads of B use
#pragma once
#include "common.cuh"

namespace b200sp {

__device__ __forceinline__ unsigned probe_hash(unsigned long long i) {
  unsigned long long z = i * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27;
  return (unsigned)(z >> 20);
}

// `gathers` independent reads of table[hash(i) & mask] (mask + 1 a power of two), eight in flight per thread, indices made in
// registers so that nothing but the gather touches memory.  ELEM = 4 or 2 bytes per entry.  SMEM: the table (at most
// smem_elems entries) is first copied into shared memory and gathered from there.
template <typename E, bool SMEM>
__global__ void __launch_bounds__(256) probe_gather_kernel(const E* __restrict__ table, unsigned mask, long long gathers,
                                                           float* __restrict__ sink) {
  extern __shared__ __align__(16) unsigned char probe_smem[];
  const E* src = table;
  if (SMEM) {
    E* t = reinterpret_cast<E*>(probe_smem);
    for (unsigned i = threadIdx.x; i <= mask; i += blockDim.x) t[i] = table[i];
    __syncthreads();
    src = t;
  }
  const long long stride = (long long)gridDim.x * blockDim.x;
  float s = 0.0f;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < gathers; i += stride * 8) {
    E v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const unsigned idx = probe_hash((unsigned long long)(i + u * stride)) & mask;
      v[u] = (i + u * stride < gathers) ? (SMEM ? src[idx] : __ldg(src + idx)) : E(0);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) s += (float)v[u];
  }
  if (s == 1.2345e-30f) *sink = s;   // keeps the loads alive; practically never true
}

// Streams `bytes` (a multiple of 16) once with coalesced 128-bit loads that do not allocate in L1.
__global__ void __launch_bounds__(256) probe_stream_kernel(const int4* __restrict__ buf, long long vecs, float* __restrict__ sink) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  int acc = 0;
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 3 * stride < vecs; i += 4 * stride) {
    const int4 a = ld_stream_i4((const int*)(buf + i)), b = ld_stream_i4((const int*)(buf + i + stride));
    const int4 c = ld_stream_i4((const int*)(buf + i + 2 * stride)), d = ld_stream_i4((const int*)(buf + i + 3 * stride));
    acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ d.x ^ d.y ^ d.z ^ d.w;
  }
  for (; i < vecs; i += stride) { const int4 a = ld_stream_i4((const int*)(buf + i)); acc ^= a.x ^ a.y ^ a.z ^ a.w; }
  if (acc == 0x5A5A1234) *sink = (float)acc;
}

// `reads` random chunks of GL * 16 bytes (GL = 8, 16 or 32 lanes: one, two or four consecutive 128-byte lines) out of a buffer of
// `chunks` such chunks (a power of two): every group of GL lanes reads one chunk, 16 bytes per lane, U chunks in flight per group
// -- the access pattern of the k-sliced SpMM kernel's reads of B (GL = 8, U = 4 in registers).  ASYNC: the chunks go to shared
// memory with cp.async (16 bytes per lane) instead of registers, so the bytes in flight are bounded by shared memory rather than
// by the register file.
template <int U, bool ASYNC, int GL>
__global__ void __launch_bounds__(256) probe_lines_kernel(const int4* __restrict__ buf, unsigned chunk_mask, long long reads,
                                                          float* __restrict__ sink) {
  extern __shared__ __align__(16) unsigned char probe_smem[];
  const long long groups = ((long long)gridDim.x * blockDim.x) / GL;
  const long long g = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / GL;
  const int l = threadIdx.x % GL;
  int acc = 0;
  int4* mine = reinterpret_cast<int4*>(probe_smem) + (size_t)threadIdx.x * U;
  for (long long i = g; i < reads; i += groups * U) {
    if (ASYNC) {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const unsigned chunk = probe_hash((unsigned long long)(i + u * groups)) & chunk_mask;
        const unsigned dst = (unsigned)__cvta_generic_to_shared(mine + u);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(buf + (size_t)chunk * GL + l) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
      for (int u = 0; u < U; ++u) { const int4 v = mine[u]; acc ^= v.x ^ v.y ^ v.z ^ v.w; }
    } else {
      int4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const unsigned chunk = probe_hash((unsigned long long)(i + u * groups)) & chunk_mask;
        v[u] = (i + u * groups < reads) ? __ldg(buf + (size_t)chunk * GL + l) : make_int4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
  }
  if (acc == 0x5A5A1234) *sink = (float)acc;
}

// The gather phase of a CSR SpMV alone: every thread streams groups of four (col, val) pairs (two groups in flight,
// grid-stride, coalesced 128-bit loads that do not allocate in L1), gathers x and adds the products into one register;
// one float per thread goes to `out`.  Launched with a given amount of dynamic shared memory that nothing uses, it shows
// what the gathers cost as a function of the L1 that the carve-out leaves: on a matrix with skewed columns (few entries of
// x take most of the gathers) that is what decides the time of an SpMV kernel.
template <typename T>
__global__ void __launch_bounds__(1024) probe_spmv_gather_kernel(const int* __restrict__ col_idx, const T* __restrict__ vals, long long quads,
                                                                const T* __restrict__ x, float* __restrict__ out) {
  float acc = 0.0f;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < quads; q += 2 * stride) {
    const int4 c0 = ld_stream_i4(col_idx + 4 * q);
    float v0[4], v1[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    ld_stream_vals4(vals + 4 * q, v0);
    const bool two = q + stride < quads;
    int4 c1 = c0;                        // a valid column when the second group does not exist (its values are zero)
    if (two) { c1 = ld_stream_i4(col_idx + 4 * (q + stride)); ld_stream_vals4(vals + 4 * (q + stride), v1); }
    const float x0 = ld_gather(x + c0.x), x1 = ld_gather(x + c0.y), x2 = ld_gather(x + c0.z), x3 = ld_gather(x + c0.w);
    const float x4 = ld_gather(x + c1.x), x5 = ld_gather(x + c1.y), x6 = ld_gather(x + c1.z), x7 = ld_gather(x + c1.w);
    acc += v0[0] * x0 + v0[1] * x1 + v0[2] * x2 + v0[3] * x3;
    if (two) acc += v1[0] * x4 + v1[1] * x5 + v1[2] * x6 + v1[3] * x7;
  }
  out[(long long)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

}  // namespace b200sp
