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

// 128-bit loads from a 32-bit shared-memory address (no generic-address arithmetic in the row loops)
__device__ __forceinline__ float4 lds128(unsigned addr, const float4*) {
  float4 r;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(addr));
  return r;
}
__device__ __forceinline__ uint4 lds128(unsigned addr, const uint4*) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
  return r;
}
__device__ __forceinline__ uint2 lds64(unsigned addr) {
  uint2 r;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(r.x), "=r"(r.y) : "r"(addr));
  return r;
}
__device__ __forceinline__ int4 lds128(unsigned addr, const int4*) {
  int4 r;
  asm volatile("ld.shared.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
  return r;
}

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

// ---- the same product with A re-laid once per call ------------------------------------------------------------
//
// In spmm_bstage_kernel above every (row, slice) pair walks the row's (col, val) pairs again, and the L1 data pipe
// that kernel is bound by spends 40 % of its wavefronts on things other than the reads of B: single steps up to the
// first multiple of four, the copies of the pairs into the per-warp buffers, and bank conflicts between the two
// (four) lane groups of a quarter warp whose rows of the slice fall into the same half (quarter) of a 128-byte bank
// line; a quarter of its lanes idle because the rows of a warp's step differ in length.  All of this depends only
// on A, so it is dealt with once per plan and once per call instead of once per slice:
//
// * per plan (quad_order_* kernels): the rows of at most kLongRow nonzeros sorted by length, longest first, in blocks
//   of GPW = 32 / LANES list slots: the rows of a block -- one step of a warp -- are equally long, except where the
//   length changes along the list; a quad is a group of four nonzeros;
// * per call (spmm_bstage_prep_kernel): A copied into two arrays of quads: four 16-bit offsets col * ROW_BYTES / 16 (the
//   slice has fewer than 2^16 sixteen-byte pieces), and the four values as stored (FP32 or BF16).  Quad i of the row in
//   slot g of block b sits at quad position pos[b] + i * GPW + g, so the GPW groups of a warp read GPW consecutive
//   quads at every step.  The last quad of a row is padded with (0, 0), which is never multiplied.  Inside a row the entries are ordered by (col - g) mod G, G = 128 / ROW_BYTES
//   rows of the slice per bank line: the groups of a quarter warp own neighbouring slots, so while the classes of
//   their rows are equally long they read different parts of the bank line.  (The order of a row's products
//   changes; each lane still adds them in one fixed order.)
//
// spmm_bstage_quads_kernel then needs no alignment steps and gets a block's quads with ONE bulk copy per array (TMA,
// on a barrier of the warp's own, outside the LSU pipe).
// Rows longer than kLongRow are left to spmm_long_row_kernel.
template <typename T, int ROW_BYTES>
__global__ void __launch_bounds__(256)
spmm_bstage_prep_kernel(int slots, int gpw, const int* __restrict__ quad_row, const int* __restrict__ quad_pos,
                        const int* __restrict__ row_ptr, const int* __restrict__ col_idx, const T* __restrict__ vals,
                        unsigned short* __restrict__ qoff, T* __restrict__ qval) {
  constexpr int G = 128 / ROW_BYTES;
  constexpr unsigned FULL = 0xFFFFFFFFu;
  grid_dependency_wait();
  const int lane = threadIdx.x & 31, sub = lane & 7, first = lane & ~7;   // eight lanes per row, four rows per warp
  const long long slot = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
  int rs = 0, re = 0, g = 0;
  long long base = 0;       // entry index of quad 0 of this row
  if (slot < slots) {
    const int row = __ldg(quad_row + slot);
    const int b = (int)(slot / gpw);
    g = (int)(slot - (long long)b * gpw);
    if (row >= 0) { rs = __ldg(row_ptr + row); re = __ldg(row_ptr + row + 1); }
    base = ((long long)__ldg(quad_pos + b) + g) * 4;
  }
  const int len = re - rs;
  const int stride = gpw * 4;                 // entries from one quad of the row to the next
  const int gc = g & (G - 1);
  int start[G];    // where class j begins inside the row
  {
    int cnt[G];
#pragma unroll
    for (int j = 0; j < G; ++j) cnt[j] = 0;
    if (G > 1) {
      for (int p = rs + sub; p < re; p += 8) {
        const int cls = (__ldg(col_idx + p) - gc) & (G - 1);
#pragma unroll
        for (int j = 0; j < G; ++j) cnt[j] += (cls == j);
      }
#pragma unroll
      for (int j = 0; j < G; ++j) {
        cnt[j] += __shfl_xor_sync(FULL, cnt[j], 1);
        cnt[j] += __shfl_xor_sync(FULL, cnt[j], 2);
        cnt[j] += __shfl_xor_sync(FULL, cnt[j], 4);
      }
    }
    int run = 0;
#pragma unroll
    for (int j = 0; j < G; ++j) { start[j] = run; run += cnt[j]; }
  }
  int longest = len;    // the ballots below need every lane of the warp: all four rows walk as far as the longest
  longest = max(longest, __shfl_xor_sync(FULL, longest, 8));
  longest = max(longest, __shfl_xor_sync(FULL, longest, 16));
  for (int p0 = 0; p0 < longest; p0 += 8) {
    const bool valid = p0 + sub < len;
    int c = 0, cls = -1;
    T v = T();
    if (valid) {
      c = __ldg(col_idx + rs + p0 + sub);
      v = __ldg(vals + rs + p0 + sub);
      cls = (c - gc) & (G - 1);
    }
    int dest = 0;
#pragma unroll
    for (int j = 0; j < G; ++j) {
      const unsigned bits = (__ballot_sync(FULL, cls == j) >> first) & 0xFFu;
      if (cls == j) dest = start[j] + __popc(bits & ((1u << sub) - 1u));
      start[j] += __popc(bits);
    }
    if (valid) {
      const long long e = base + (long long)(dest >> 2) * stride + (dest & 3);
      qoff[e] = (unsigned short)(c * (ROW_BYTES / 16));
      qval[e] = v;
    }
  }
  for (int d = len + sub; d < ((len + 3) & ~3); d += 8) {
    const long long e = base + (long long)(d >> 2) * stride + (d & 3);
    qoff[e] = 0;
    qval[e] = T();
  }
}

// One quad of the re-laid A: the shared-memory addresses of this lane's piece of the four rows of the slice, and the four values.
template <typename T, bool SHARED> struct QuadLoad;
template <bool SHARED> struct QuadLoad<float, SHARED> {
  static __device__ __forceinline__ void ld(const uint2* qo, const float* qv, unsigned so, unsigned sv, unsigned bs, unsigned (&a)[4], float (&v)[4]) {
    const uint2 o = SHARED ? lds64(so) : __ldg(qo);
    const float4 x = SHARED ? lds128(sv, (const float4*)nullptr) : __ldg((const float4*)qv);
    a[0] = bs + ((o.x & 0xFFFFu) << 4); a[1] = bs + ((o.x >> 16) << 4); a[2] = bs + ((o.y & 0xFFFFu) << 4); a[3] = bs + ((o.y >> 16) << 4);
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
  }
};
template <bool SHARED> struct QuadLoad<bf16_t, SHARED> {
  static __device__ __forceinline__ void ld(const uint2* qo, const bf16_t* qv, unsigned so, unsigned sv, unsigned bs, unsigned (&a)[4], float (&v)[4]) {
    const uint2 o = SHARED ? lds64(so) : __ldg(qo);
    const uint2 x = SHARED ? lds64(sv) : __ldg((const uint2*)qv);
    a[0] = bs + ((o.x & 0xFFFFu) << 4); a[1] = bs + ((o.x >> 16) << 4); a[2] = bs + ((o.y & 0xFFFFu) << 4); a[3] = bs + ((o.y >> 16) << 4);
    v[0] = __uint_as_float(x.x << 16); v[1] = __uint_as_float(x.x & 0xFFFF0000u);
    v[2] = __uint_as_float(x.y << 16); v[3] = __uint_as_float(x.y & 0xFFFF0000u);
  }
};

// acc += the products of one row's quads 0 .. (len + 3) / 4 - 1 with this lane's columns of the slice (whose piece of row 0
// is at shared address bs).  SHARED: the quads sit in shared memory at addresses so / sv, else in global memory at qo / qv;
// consecutive quads of the row are qstride quads apart.
template <typename T, int VEC, bool SHARED>
__device__ __forceinline__ void bstage_row_quads(const uint2* __restrict__ qo, const T* __restrict__ qv, unsigned so, unsigned sv, int qstride,
                                                 int len, unsigned bs, float (&acc)[VEC], float (&tot)[VEC]) {
  typedef typename RawVec<T, VEC>::type raw_t;
  const int full = len >> 2, rem = len & 3;
  int fold = 0;
  for (int i = 0; i < full; ++i) {
    if (++fold > kChainBlock / 4) {
      fold = 1;
#pragma unroll
      for (int j = 0; j < VEC; ++j) { tot[j] += acc[j]; acc[j] = 0.0f; }
    }
    unsigned a[4];
    float v[4];
    QuadLoad<T, SHARED>::ld(qo, qv, so, sv, bs, a, v);
    so += 8u * qstride; sv += 4u * (unsigned)sizeof(T) * qstride; qo += qstride; qv += 4 * qstride;
    raw_t b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) b[u] = lds128(a[u], (const raw_t*)nullptr);
#pragma unroll
    for (int u = 0; u < 4; ++u) RawVec<T, VEC>::fma_mixed(b[u], v[u], acc);
  }
  if (rem) {   // the padded last quad: its padding is never multiplied (0 * inf would be NaN)
    unsigned a[4];
    float v[4];
    QuadLoad<T, SHARED>::ld(qo, qv, so, sv, bs, a, v);
    RawVec<T, VEC>::fma_mixed(lds128(a[0], (const raw_t*)nullptr), v[0], acc);
    if (rem > 1) RawVec<T, VEC>::fma_mixed(lds128(a[1], (const raw_t*)nullptr), v[1], acc);
    if (rem > 2) RawVec<T, VEC>::fma_mixed(lds128(a[2], (const raw_t*)nullptr), v[2], acc);
  }
}

// Dynamic shared memory: [ slice of B: bslice_bytes | per warp: capq offset quads (8 B each), capq value quads (4 values each) ]; capq is even.
// CTA `chunk` of a slice takes the blocks chunk, chunk + row_chunks, ... of the sorted list, its warps in turn, so that
// every CTA gets the same mix of long and short rows.  A block of more than capq quads is read from global memory.
// (Fetching the next block's quads a step ahead into a second half of the buffer was measured: no gain.)
template <typename T, int VEC, int LANES, int THREADS>
__global__ void __launch_bounds__(THREADS)
spmm_bstage_quads_kernel(const __grid_constant__ CUtensorMap tmapB, int n, int k, int row_chunks, int blocks, int box_rows, int bslice_bytes,
                         int capq, const int* __restrict__ quad_row, const int* __restrict__ quad_len, const int* __restrict__ quad_pos,
                         const unsigned short* __restrict__ qoff, const T* __restrict__ qval, T* __restrict__ Y, float alpha, float beta,
                         int* __restrict__ err, int spin_limit, int no_copies) {
  constexpr int KS = LANES * VEC, ROW_BYTES = LANES * 16, GPW = 32 / LANES, WARPS = THREADS / 32;
  constexpr unsigned FULL = 0xFFFFFFFFu;
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long bar;
  __shared__ __align__(8) unsigned long long wbar[WARPS];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int slice = blockIdx.x / row_chunks, chunk = blockIdx.x - slice * row_chunks;
  const int col_base = slice * KS;
  if (tid == 0) mbar_init(smem_addr(&bar), 1);
  if (lane == 0) mbar_init(smem_addr(&wbar[warp]), 1);
  mbar_init_fence();
  __syncthreads();
  grid_dependency_wait();   // nothing above touches global memory
  if (tid == 0 && !no_copies) {   // no_copies (a test switch): nothing is issued, the wait below runs out with nothing in flight
    const int boxes = (n + box_rows - 1) / box_rows;
    mbar_arrive_expect_tx(smem_addr(&bar), (unsigned)boxes * (unsigned)box_rows * ROW_BYTES);   // rows past n are zero-filled and still counted
    for (int b = 0; b < boxes; ++b)
      tma_load_2d(smem_addr(smem + (size_t)b * box_rows * ROW_BYTES), &tmapB, col_base, b * box_rows, smem_addr(&bar));
  }
  const int gl = lane / LANES, l = lane % LANES;     // group inside the warp, lane inside the group
  const int col0 = col_base + l * VEC;
  const bool active = col0 < k;
  const unsigned bs = smem_addr(smem) + l * 16;
  constexpr unsigned VQ = 4u * (unsigned)sizeof(T);                          // bytes of a quad's values
  const unsigned woff = smem_addr(smem) + bslice_bytes + warp * capq * (8u + VQ);   // the warp's buffer: capq quads of offsets, then of values
  const unsigned wval = woff + capq * 8u;
  const unsigned my_bar = smem_addr(&wbar[warp]);
  const long long step_blocks = (long long)WARPS * row_chunks;
  // one step's description, a value per lane: lanes < GPW the row number (m_row) and length (m_len) of their slot,
  // lanes 30 / 31 the block's last / first quad position (m_len)
  auto load_meta = [&](long long b, int& m_row, int& m_len) {
    m_row = -1; m_len = 0;
    if (b < blocks) {
      if (lane < GPW) { m_row = __ldg(quad_row + b * GPW + lane); m_len = __ldg(quad_len + b * GPW + lane); }
      else if (lane >= 30) m_len = __ldg(quad_pos + b + (31 - lane));
    }
  };
  // the bulk copies that fetch a block's quads (lane 0 issues; the buffer must be free)
  auto issue = [&](int q0, int nq) {
    if (nq > 0 && nq <= capq && lane == 0) {
      mbar_arrive_expect_tx(my_bar, (unsigned)nq * (8u + VQ));
      bulk_copy_g2s(woff, qoff + (long long)q0 * 4, (unsigned)nq * 8u, my_bar);
      bulk_copy_g2s(wval, qval + (long long)q0 * 4, (unsigned)nq * VQ, my_bar);
    }
  };
  long long b = chunk + (long long)warp * row_chunks;
  int row_cur, len_cur, row_next, len_next;
  load_meta(b, row_cur, len_cur);
  load_meta(b + step_blocks, row_next, len_next);
  int q0_cur = __shfl_sync(FULL, len_cur, 31), nq_cur = __shfl_sync(FULL, len_cur, 30) - q0_cur;
  issue(q0_cur, nq_cur);        // the copies of the first step overlap the fetch of the slice of B (no block: nq_cur is 0)
  unsigned phase = 0;
  const bool arrived = mbar_wait_bounded(smem_addr(&bar), 0, spin_limit);
  if (!__syncthreads_and(arrived)) {
    if (tid == 0) atomicExch(err, 1);
    (void)mbar_wait_bounded(smem_addr(&bar), 0, spin_limit);   // bounded second chance for the copies in flight
    if (nq_cur > 0 && nq_cur <= capq) (void)mbar_wait_bounded(my_bar, 0, spin_limit);
    return;
  }
  for (; b < blocks; b += step_blocks) {
    const int q0_next = __shfl_sync(FULL, len_next, 31), nq_next = __shfl_sync(FULL, len_next, 30) - q0_next;
    const bool staged = nq_cur > 0 && nq_cur <= capq;
    if (staged) {
      const bool ok = mbar_wait_bounded(my_bar, phase, spin_limit);
      if (!__all_sync(FULL, ok)) {
        if (lane == 0) atomicExch(err, 1);
        (void)mbar_wait_bounded(my_bar, phase, spin_limit);
        return;
      }
      phase ^= 1u;
    }
    const int row = __shfl_sync(FULL, row_cur, gl), len = __shfl_sync(FULL, len_cur, gl);
    float acc[VEC], tot[VEC];   // acc: the current block of at most kChainBlock products; tot: the sum of the completed blocks
#pragma unroll
    for (int j = 0; j < VEC; ++j) { acc[j] = 0.0f; tot[j] = 0.0f; }
    if (staged) {
      bstage_row_quads<T, VEC, true>(nullptr, nullptr, woff + 8u * gl, wval + VQ * gl, GPW, len, bs, acc, tot);
    } else {
      bstage_row_quads<T, VEC, false>((const uint2*)qoff + q0_cur + gl, qval + 4LL * (q0_cur + gl), 0u, 0u, GPW, len, bs, acc, tot);
    }
    __syncwarp();                       // every lane is done with the buffer: the next block's quads may land in it
    issue(q0_next, nq_next);            // (past the last block nq_next is 0)
    if (active && row >= 0) {
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
    row_cur = row_next; len_cur = len_next; q0_cur = q0_next; nq_cur = nq_next;
    load_meta(b + 2 * step_blocks, row_next, len_next);
  }
}

}  // namespace b200sp
