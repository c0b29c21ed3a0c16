// Host side of libb200sp.so: SpMM kernel selection and launches.
// One of the pieces of the single translation unit b200sp.cu; include/b200sp.h states the contract of every entry point.
#pragma once
#include "host_spmv.cuh"
#include "spmm_kernels.cuh"
#include "spmm_bstage_kernels.cuh"
#include "format_kernels.cuh"

namespace {

// Rows of at most kLongRow nonzeros by one lane group each; longer rows by a CTA per (row, 8 * VEC columns).
template <typename T, int VEC, int LANES, int NCH>
int launch_spmm(b200sp_plan* p, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y, float alpha, float beta,
                cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  constexpr int GROUPS = kSpmmThreads / LANES;
  const unsigned grid = (unsigned)((I.m + GROUPS - 1) / GROUPS);
  tl_pdl_kernel = true;
  int rc = launch(spmm_row_group_kernel<T, VEC, LANES, NCH, kSpmmThreads>, dim3(grid), dim3(kSpmmThreads), stream, B,
                  (size_t)I.n * k * sizeof(T), dev, (int)I.m, k, p->row_ptr, col_idx, vals, B, Y, alpha, beta, kLongRow);
  if (rc != B200SP_OK || p->num_long == 0) return rc;
  const long long ctas = (long long)((k + 8 * VEC - 1) / (8 * VEC)) * p->num_long;
  if (ctas >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  tl_pdl_kernel = true;
  return launch(spmm_long_row_kernel<T, VEC, kSpmmThreads>, dim3((unsigned)ctas), dim3(kSpmmThreads), stream, nullptr, 0, dev, k, p->num_long,
                (const int*)p->long_rows, p->row_ptr, col_idx, vals, B, Y, alpha, beta);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn tensor_map_encoder() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    else
      (void)cudaGetLastError();
  }
  return fn;
}

// B slice in shared memory: used when A has few enough columns and every row of B is re-used often enough.
template <typename T, int VEC, int LANES, int THREADS = 1024>
int launch_spmm_bstage(b200sp_plan* p, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y, float alpha, float beta,
                       cudaStream_t stream, DeviceInfo* dev, EncodeTiledFn encode) {
  const b200sp_plan_info_t& I = p->info;
  constexpr int KS = LANES * VEC, ROW_BYTES = LANES * 16;
  const int box_rows = I.n < 256 ? (int)I.n : 256;
  const int boxes = (int)((I.n + box_rows - 1) / box_rows);
  const size_t bslice = (((size_t)boxes * box_rows * ROW_BYTES) + 127) & ~(size_t)127;
  // what the slice of B leaves of the SM's shared memory is split among the warps as staging buffers for their (col, val) pairs
  const size_t limit = (size_t)kSmemPerSm - 2048;
  int capw = 0;
  if (g_opt.bstage_stage_a && bslice < limit) {
    const size_t per_warp = (limit - bslice) / (THREADS / 32);
    const long long entries = (long long)(per_warp / (4 + sizeof(T))) & ~7LL;
    if (entries >= 72) capw = (int)(entries > 4096 ? 4096 : entries) - 4;
  }
  const size_t smem = bslice + (capw > 0 ? (size_t)(THREADS / 32) * (capw + 4) * (4 + sizeof(T)) : 0);
  CUtensorMap map;
  const cuuint64_t gdim[2] = {(cuuint64_t)k, (cuuint64_t)I.n};
  const cuuint64_t gstride[1] = {(cuuint64_t)k * sizeof(T)};
  const cuuint32_t box[2] = {(cuuint32_t)KS, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult cr = encode(&map, sizeof(T) == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<T*>(B), gdim,
                             gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return B200SP_ERR_UNSUPPORTED;
  auto kernel = spmm_bstage_kernel<T, VEC, LANES, THREADS>;
  static bool configured[64] = {};
  if (!configured[p->device]) {
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerSm - 2048));
    configured[p->device] = true;
  }
  const int slices = (k + KS - 1) / KS;
  const int per_cta = g_opt.bstage_nnz > 0 ? g_opt.bstage_nnz : 131072;
  long long chunks = (I.nnz + per_cta - 1) / per_cta;   // a given number of nonzeros per CTA ...
  const long long fill = (2LL * dev->sms + slices - 1) / slices;   // ... but at least two CTAs per SM over the grid
  if (chunks < fill) chunks = fill;
  if (chunks > I.m) chunks = I.m;
  if (chunks < 1) chunks = 1;
  const int rows_per_chunk = (int)((I.m + chunks - 1) / chunks);
  const int row_chunks = (int)((I.m + rows_per_chunk - 1) / rows_per_chunk);
  if ((long long)slices * row_chunks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  int rc = ensure_err_flag(dev);
  if (rc != B200SP_OK) return rc;
  tl_pdl_kernel = true;
  return launch_smem(kernel, dim3((unsigned)(slices * row_chunks)), dim3(THREADS), smem, stream, nullptr, 0, dev, map, (int)I.m, (int)I.n,
                     k, row_chunks, rows_per_chunk, box_rows, (int)bslice, capw, p->row_ptr, col_idx, vals, Y, alpha, beta, dev->err_flag,
                     g_opt.spin_limit, g_opt.debug_no_copies);
}

// Exclusive scan of `count` ints in place; bsum: (count + kScanBlock - 1) / kScanBlock + 1 ints of scratch.  Three launches.
int device_scan_in_place(int* data, long long count, int* bsum, cudaStream_t stream) {
  const long long blocks = (count + kScanBlock - 1) / kScanBlock;
  if (blocks < 1 || blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  scan_block_sums_kernel<<<(unsigned)blocks, 256, 0, stream>>>(data, count, bsum);
  plan_compact_scan_kernel<<<1, 1024, 0, stream>>>(bsum, (int)blocks);
  scan_apply_kernel<<<(unsigned)blocks, 256, 0, stream>>>(data, count, bsum, data);
  g_launches += 3;
  CU(cudaGetLastError());
  return B200SP_OK;
}

// The processing order of spmm_bstage_quads_kernel (see plan_kernels.cuh), built once per plan and lane-group width, on the
// device and in stream order: no synchronisation.  B200SP_ERR_UNSUPPORTED when the positions would not fit 32 bits.
int plan_quad_order(b200sp_plan* p, int gpw, cudaStream_t stream, DeviceInfo* dev) {
  static_assert(kLongRow == 1024, "quad_key() assumes rows of at most 1024 nonzeros");
  if (p->quad_block && p->quad_gpw == gpw) return B200SP_OK;
  const b200sp_plan_info_t& I = p->info;
  const long long listed = I.m - p->num_long;
  const long long blocks = (listed + gpw - 1) / gpw;
  if ((I.nnz + 3 * I.m) / 4 + (long long)(kLongRow / 4 + 2) * gpw >= (1LL << 31) - 64 || blocks < 1) return B200SP_ERR_UNSUPPORTED;
  if (p->quad_block) { CU(cudaFreeAsync(p->quad_block, stream)); p->quad_block = nullptr; p->quad_gpw = 0; }
  long long rows_per_blk = (I.m + 65535) / 65536;
  if (rows_per_blk < 256) rows_per_blk = 256;
  rows_per_blk = (rows_per_blk + 31) / 32 * 32;
  const long long nblk = (I.m + rows_per_blk - 1) / rows_per_blk;
  const long long slots = blocks * gpw, table = (long long)kQuadKeys * nblk;
  const long long scan_len = table > blocks + 1 ? table : blocks + 1;
  auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
  const size_t o_row = 0, o_len = up((size_t)slots * 4), o_pos = o_len + up((size_t)slots * 4), keep = o_pos + up((size_t)(blocks + 1) * 4);
  void* blk = nullptr;
  void* tmp = nullptr;      // the histogram table and the scan's block sums: only needed while the order is built
  int rc = pool_alloc(dev, &blk, keep, stream);
  if (rc != B200SP_OK) return rc;
  rc = pool_alloc(dev, &tmp, up((size_t)table * 4) + up((size_t)(scan_len / kScanBlock + 2) * 4), stream);
  if (rc != B200SP_OK) { cudaFreeAsync(blk, stream); return rc; }
  int* row_of = (int*)((char*)blk + o_row);
  int* len_of = (int*)((char*)blk + o_len);
  int* pos = (int*)((char*)blk + o_pos);
  int* hist = (int*)tmp;
  int* bsum = (int*)((char*)tmp + up((size_t)table * 4));
  auto fail = [&](int code) { cudaFreeAsync(tmp, stream); cudaFreeAsync(blk, stream); return code; };
#define CUQ(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(cuda_fail(e_, #call)); } while (0)
  CUQ(cudaMemsetAsync(row_of, 0xFF, (size_t)slots * 4, stream));      // unused slots: row -1, length 0
  CUQ(cudaMemsetAsync(len_of, 0, (size_t)slots * 4, stream));
  const unsigned grid = (unsigned)((nblk + 3) / 4);
  quad_order_hist_kernel<<<grid, 128, 0, stream>>>(p->row_ptr, (int)I.m, (int)rows_per_blk, (int)nblk, hist);
  g_launches++;
  CUQ(cudaGetLastError());
  rc = device_scan_in_place(hist, table, bsum, stream);
  if (rc != B200SP_OK) return fail(rc);
  quad_order_scatter_kernel<<<grid, 128, 0, stream>>>(p->row_ptr, (int)I.m, (int)rows_per_blk, (int)nblk, hist, row_of, len_of);
  quad_order_block_quads_kernel<<<(unsigned)((blocks + 1 + 255) / 256), 256, 0, stream>>>(len_of, (int)blocks, gpw, pos);
  g_launches += 2;
  CUQ(cudaGetLastError());
  rc = device_scan_in_place(pos, blocks + 1, bsum, stream);
  if (rc != B200SP_OK) return fail(rc);
  CUQ(cudaFreeAsync(tmp, stream));
#undef CUQ
  p->quad_block = blk;
  p->quad_row = row_of;
  p->quad_len = len_of;
  p->quad_pos = pos;
  p->quad_gpw = gpw;
  p->quad_blocks = (int)blocks;
  return B200SP_OK;
}

// The same with the rows in the plan's sorted order and A re-laid once per call into padded quads (spmm_bstage_prep_kernel),
// which the main kernel's warps fetch with bulk copies; rows longer than kLongRow by spmm_long_row_kernel.
template <typename T, int VEC, int LANES, int THREADS = 1024>
int launch_spmm_bstage_quads(b200sp_plan* p, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y, float alpha, float beta,
                             cudaStream_t stream, DeviceInfo* dev, EncodeTiledFn encode) {
  const b200sp_plan_info_t& I = p->info;
  constexpr int KS = LANES * VEC, ROW_BYTES = LANES * 16, GPW = 32 / LANES, WARPS = THREADS / 32;
  const int box_rows = I.n < 256 ? (int)I.n : 256;
  const int boxes = (int)((I.n + box_rows - 1) / box_rows);
  const size_t bslice = (((size_t)boxes * box_rows * ROW_BYTES) + 127) & ~(size_t)127;
  // what the slice of B leaves of the SM's shared memory is split among the warps as buffers for their blocks' quads
  // (four 16-bit offsets and four values each)
  constexpr size_t QUAD_BYTES = 8 + 4 * sizeof(T);
  const size_t limit = (size_t)kSmemPerSm - 2048 - 32 * WARPS;
  int capq = 0;
  if (g_opt.bstage_stage_a && bslice < limit) {
    const size_t quads = (limit - bslice) / WARPS / QUAD_BYTES;
    capq = (int)(quads > 2048 ? 2048 : quads) & ~1;
    if (capq < 2 * GPW) capq = 0;
  }
  const size_t smem = bslice + (((size_t)WARPS * capq * QUAD_BYTES + 15) & ~(size_t)15);
  CUtensorMap map;
  const cuuint64_t gdim[2] = {(cuuint64_t)k, (cuuint64_t)I.n};
  const cuuint64_t gstride[1] = {(cuuint64_t)k * sizeof(T)};
  const cuuint32_t box[2] = {(cuuint32_t)KS, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult cr = encode(&map, sizeof(T) == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<T*>(B), gdim,
                             gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return B200SP_ERR_UNSUPPORTED;
  int rc = plan_quad_order(p, GPW, stream, dev);
  if (rc != B200SP_OK) return rc;
  auto kernel = spmm_bstage_quads_kernel<T, VEC, LANES, THREADS>;
  static bool configured[64] = {};
  if (!configured[p->device]) {
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerSm - 2048));
    configured[p->device] = true;
  }
  const int slices = (k + KS - 1) / KS;
  const int blocks = p->quad_blocks;
  const long long most = (blocks + WARPS - 1) / WARPS;   // a block per warp at least
  long long chunks;
  if (g_opt.bstage_nnz > 0) {
    chunks = (I.nnz + g_opt.bstage_nnz - 1) / g_opt.bstage_nnz;   // a given number of nonzeros per CTA ...
    const long long fill = (2LL * dev->sms + slices - 1) / slices;   // ... but at least two CTAs per SM over the grid
    if (chunks < fill) chunks = fill;
  } else {
    // One CTA per SM is resident and all CTAs take the same time (each gets the same mix of rows), so the kernel lasts
    // ceil(CTAs / SMs) rounds of (nonzeros per CTA + the fetch of the slice of B, about 4096 nonzeros' worth): the chunk
    // count with the smallest product, among those that leave a CTA at least 8192 nonzeros (or one chunk).
    chunks = 1;
    double best = 0.0;
    for (long long c = 1; c <= 4096 && c <= most && (c == 1 || I.nnz / c >= 8192); ++c) {
      const double rounds = (double)((slices * c + dev->sms - 1) / dev->sms);
      const double cost = rounds * ((double)I.nnz / (double)c + 4096.0);
      if (c == 1 || cost < best) { best = cost; chunks = c; }
    }
  }
  if (chunks > most) chunks = most;
  if (chunks < 1) chunks = 1;
  const int row_chunks = (int)chunks;
  if ((long long)slices * row_chunks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  rc = ensure_err_flag(dev);
  if (rc != B200SP_OK) return rc;
  // the per-call copy of A: at most the rows' quads plus (kLongRow / 4 + 2) * GPW of padding where the length changes along the list
  const size_t entries = (((size_t)((I.nnz + 3 * I.m) / 4) + (size_t)(kLongRow / 4 + 2) * GPW) * 4 + 15) & ~(size_t)7;
  void* scratch = nullptr;
  rc = pool_alloc(dev, &scratch, entries * (2 + sizeof(T)), stream);
  if (rc != B200SP_OK) return rc;
  unsigned short* qoff = (unsigned short*)scratch;       // entries 16-bit offsets, then entries values (16-byte aligned: entries is a multiple of 8)
  T* qval = (T*)((char*)scratch + entries * 2);
  const long long slots = (long long)blocks * GPW;
  tl_pdl_kernel = true;
  rc = launch(spmm_bstage_prep_kernel<T, ROW_BYTES>, dim3((unsigned)((slots * 8 + 255) / 256)), dim3(256), stream, nullptr, 0, dev, (int)slots, GPW,
              (const int*)p->quad_row, (const int*)p->quad_pos, p->row_ptr, col_idx, vals, qoff, qval);
  if (rc == B200SP_OK) {
    tl_pdl_kernel = true;
    rc = launch_smem(kernel, dim3((unsigned)(slices * row_chunks)), dim3(THREADS), smem, stream, nullptr, 0, dev, map, (int)I.n, k, row_chunks,
                     blocks, box_rows, (int)bslice, capq, (const int*)p->quad_row, (const int*)p->quad_len, (const int*)p->quad_pos,
                     (const unsigned short*)qoff, (const T*)qval, Y, alpha, beta, dev->err_flag, g_opt.spin_limit, g_opt.debug_no_copies);
  }
  const cudaError_t e = cudaFreeAsync(scratch, stream);
  if (e != cudaSuccess && rc == B200SP_OK) rc = cuda_fail(e, "cudaFreeAsync");
  if (rc == B200SP_OK && p->num_long > 0) {
    const long long ctas = (long long)((k + 8 * VEC - 1) / (8 * VEC)) * p->num_long;
    if (ctas >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
    tl_pdl_kernel = true;
    rc = launch(spmm_long_row_kernel<T, VEC, kSpmmThreads>, dim3((unsigned)ctas), dim3(kSpmmThreads), stream, nullptr, 0, dev, k, p->num_long,
                (const int*)p->long_rows, p->row_ptr, col_idx, vals, B, Y, alpha, beta);
  }
  return rc;
}

// Column ranges for the k-sliced kernel: how many, and the per-row cut positions (computed once per col_idx; one small
// kernel and one synchronisation of the stream).  Returns 1 in *ranges when the ranges do not apply: B's slice fits L2,
// the rows' columns are not in ascending order, or the switch says so.
int spmm_column_ranges(b200sp_plan* p, const int32_t* col_idx, int slice_bytes, cudaStream_t stream, DeviceInfo* dev, int* ranges) {
  const b200sp_plan_info_t& I = p->info;
  *ranges = 1;
  int want = g_opt.spmm_ranges;
  if (want == 0) {
    // a range of B (n / ranges rows of slice_bytes) should take at most this share of L2: the L2 of this part keeps a line
    // read by all SMs in both of its halves, and the streams of A and Y pass through it as well
    const double budget = 0.3 * (double)dev->l2_bytes;
    want = (int)(((double)I.n * slice_bytes + budget - 1) / budget);
    if (want > 8) want = 8;
  }
  if (want <= 1 || I.n < want || I.m < 1) return B200SP_OK;
  if (p->cuts_col_idx == (const void*)col_idx && p->cuts_ranges == want) { if (p->cols_sorted) *ranges = want; return B200SP_OK; }
  if (p->cuts_block) { CU(cudaFreeAsync(p->cuts_block, stream)); p->cuts_block = nullptr; p->cuts_ranges = 0; p->cuts_col_idx = nullptr; }
  const size_t bytes = (size_t)(want - 1) * (size_t)I.m * 4 + 256;
  void* blk = nullptr;
  int rc = pool_alloc(dev, &blk, bytes, stream);
  if (rc != B200SP_OK) return rc;
  int* flag = (int*)((char*)blk + (size_t)(want - 1) * (size_t)I.m * 4);
  int h = 0;
  cudaError_t e = cudaMemsetAsync(flag, 0, sizeof(int), stream);
  if (e == cudaSuccess) {
    spmm_range_cuts_kernel<<<(unsigned)((I.m + 255) / 256), 256, 0, stream>>>((int)I.m, (int)I.n, want, p->row_ptr, col_idx, (int*)blk, flag);
    g_launches++;
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&h, flag, sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) { cudaFreeAsync(blk, stream); return cuda_fail(e, "column ranges"); }
  p->cuts_block = blk;
  p->cuts_col_idx = col_idx;
  p->cuts_ranges = want;
  p->cols_sorted = h == 0;
  if (p->cols_sorted) *ranges = want;
  return B200SP_OK;
}

// nnz-balanced SpMM (spmm_flat_kernel) for matrices whose rows are too uneven for one lane group per row.
constexpr int kFlatChunk = 32;                          // nonzeros per lane group
constexpr int kFlatTile = (kSpmmThreads / 8) * kFlatChunk;   // nonzeros per CTA

bool spmm_rows_are_uneven(const b200sp_plan_info_t& I) {
  if (I.nnz <= 0 || I.m <= 0) return false;
  const int64_t nonempty = I.m - I.bin_rows[0];
  const double mean = (double)I.nnz / (double)(nonempty > 0 ? nonempty : 1);
  return (I.bin_nnz[4] + I.bin_nnz[5]) * 20 >= I.nnz      // 5 % or more of the nonzeros sit in rows longer than 128
         || I.bin_rows[0] * 4 >= I.m                        // a quarter or more of the rows are empty
         || (double)I.max_row_len > 4.0 * mean + 8.0;       // or the longest row is far above the mean
}

template <typename T, int VEC>
int run_spmm_flat(b200sp_plan* p, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y, float alpha, float beta,
                  cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  constexpr int KS = 8 * VEC;
  const int tiles = (int)((I.nnz + kFlatTile - 1) / kFlatTile);
  const int slices = (k + KS - 1) / KS;
  if ((long long)slices * tiles >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  int rc;
  if (I.bin_rows[0] > 0) {   // the rows that have nonzeros, listed once per plan (stream order, no synchronisation)
    rc = plan_compact_rows(p, stream, dev);
    if (rc != B200SP_OK) return rc;
  }
  const int rows = I.bin_rows[0] > 0 ? p->compact_rows : (int)I.m;
  const int* rp = I.bin_rows[0] > 0 ? p->compact_row_ptr : p->row_ptr;
  const int* rid = I.bin_rows[0] > 0 ? p->compact_row_id : nullptr;
  if (!p->flat_tile_row) {   // tile starts: once per plan, a small kernel in stream order
    rc = pool_alloc(dev, (void**)&p->flat_tile_row, (size_t)(tiles + 1) * sizeof(int32_t), stream);
    if (rc != B200SP_OK) return rc;
    rc = launch(plan_nnz_tile_rows_kernel, dim3((unsigned)((tiles + 1 + 255) / 256)), dim3(256), stream, nullptr, 0, dev, rp, rows,
                (int)I.nnz, kFlatTile, tiles, (int*)p->flat_tile_row);
    if (rc != B200SP_OK) return rc;
  }
  // per-call scratch: what each tile leaves unfinished and what it finishes for an earlier tile, KS floats per (slice, tile)
  float* scratch = nullptr;
  const size_t per = (size_t)slices * tiles * KS;
  rc = pool_alloc(dev, (void**)&scratch, 2 * per * sizeof(float), stream);
  if (rc != B200SP_OK) return rc;
  if (I.bin_rows[0] > 0) {
    long long blocks = ((long long)I.m * (k / VEC) + 255) / 256;
    if (blocks > (long long)dev->sms * 16) blocks = (long long)dev->sms * 16;
    rc = launch(spmm_empty_rows_kernel<T, VEC>, dim3((unsigned)blocks), dim3(256), stream, nullptr, 0, dev, (int)I.m, k, p->row_ptr, Y, beta);
  }
  if (rc == B200SP_OK) {
    tl_pdl_kernel = true;
    rc = launch(spmm_flat_kernel<T, VEC, kSpmmThreads, kFlatChunk>, dim3((unsigned)(slices * tiles)), dim3(kSpmmThreads), stream, B,
                (size_t)I.n * k * sizeof(T), dev, rows, (int)I.nnz, k, tiles, rp, rid, (const int*)p->flat_tile_row, col_idx, vals, B, Y,
                scratch, scratch + per, alpha, beta);
  }
  if (rc == B200SP_OK && tiles > 1) {
    const long long groups = (long long)slices * tiles;
    tl_pdl_kernel = true;
    rc = launch(spmm_flat_fixup_kernel<T, VEC, kSpmmThreads, kFlatTile>, dim3((unsigned)((groups * 8 + kSpmmThreads - 1) / kSpmmThreads)),
                dim3(kSpmmThreads), stream, nullptr, 0, dev, rows, (int)I.nnz, k, tiles, slices, rp, rid, (const int*)p->flat_tile_row,
                (const float*)scratch, (const float*)(scratch + per), Y, alpha, beta);
  }
  const cudaError_t e = cudaFreeAsync(scratch, stream);
  if (e != cudaSuccess && rc == B200SP_OK) rc = cuda_fail(e, "cudaFreeAsync");
  return rc;
}

template <typename T, int VEC>
int run_spmm(b200sp_plan* p, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y, float alpha, float beta,
             cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  if (I.m == 0) return B200SP_OK;
  if (alpha == 0.0f || I.nnz == 0) return run_scale<T>((long long)I.m * k, Y, beta, stream, dev);
  if (k == 1) return run_spmv<T>(p, col_idx, vals, B, Y, alpha, beta, stream, dev);   // one column: the SpMV kernels
  if (k % VEC == 0 && g_opt.spmm_bstage && I.nnz >= 4 * I.n && ((size_t)k * sizeof(T)) % 16 == 0) {
    // widest slice of B (128, 64 or 32 bytes per row) whose n rows fit in one SM's shared memory
    const size_t budget = (size_t)kSmemPerSm - 4096;
    const size_t n_pad = (size_t)((I.n + 255) / 256) * 256;
    EncodeTiledFn encode = tensor_map_encoder();
    if (encode && n_pad * 32 <= budget) {
      int rc;
#define B200SP_BSTAGE(FN)                                                                                                                  \
  do {                                                                                                                                     \
    if (g_opt.bstage_threads == 256) {                                                                                                     \
      if (n_pad * 128 <= budget) rc = FN<T, VEC, 8, 256>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                     \
      else if (n_pad * 64 <= budget) rc = FN<T, VEC, 4, 256>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                 \
      else rc = FN<T, VEC, 2, 256>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                                           \
    } else if (g_opt.bstage_threads == 512) {                                                                                              \
      if (n_pad * 128 <= budget) rc = FN<T, VEC, 8, 512>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                     \
      else if (n_pad * 64 <= budget) rc = FN<T, VEC, 4, 512>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                 \
      else rc = FN<T, VEC, 2, 512>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                                           \
    } else {                                                                                                                               \
      if (n_pad * 128 <= budget) rc = FN<T, VEC, 8, 1024>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                    \
      else if (n_pad * 64 <= budget) rc = FN<T, VEC, 4, 1024>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                \
      else rc = FN<T, VEC, 2, 1024>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);                                          \
    }                                                                                                                                      \
  } while (0)
      if (g_opt.bstage_quads) B200SP_BSTAGE(launch_spmm_bstage_quads);
      else B200SP_BSTAGE(launch_spmm_bstage);
#undef B200SP_BSTAGE
      if (rc != B200SP_ERR_UNSUPPORTED) return rc;   // unsupported shape for the tensor map: fall through to the sliced kernel
    }
  }
  if (k % VEC == 0 && g_opt.spmm_sliced) {
    // lanes per row: eight (a 128-byte slice) unless k is narrower than that
    const int vecs_k = k / VEC;
    const int lanes = vecs_k >= 8 ? 8 : (vecs_k > 2 ? 4 : vecs_k);
    const int KS = lanes * VEC, GROUPS = kSpmmThreads / lanes;
    const int slices = (k + KS - 1) / KS;
    const int row_blocks = (int)((I.m + GROUPS - 1) / GROUPS);
    if ((long long)slices * row_blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
    if (lanes == 8 && (g_opt.spmm_flat == 1 || (g_opt.spmm_flat == 2 && spmm_rows_are_uneven(I))))
      return run_spmm_flat<T, VEC>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
    int rc;
    const int mid_blocks = (p->num_medium + GROUPS - 1) / GROUPS;
    int ranges = 1;
    if (lanes == 8) {
      rc = spmm_column_ranges(p, col_idx, 8 * 16, stream, dev, &ranges);
      if (rc != B200SP_OK) return rc;
    }
    if (ranges > 1) {
      // one launch per column range; FP32 partial sums for BF16 storage come from the pool and go back in stream order
      float* partial = nullptr;
      if (sizeof(T) == 2) {
        rc = pool_alloc(dev, (void**)&partial, (size_t)I.m * (size_t)k * sizeof(float), stream);
        if (rc != B200SP_OK) return rc;
      }
      for (int r = 0; r < ranges && rc == B200SP_OK; ++r) {
        tl_pdl_kernel = true;
        rc = launch(spmm_slice_range_kernel<T, VEC, kSpmmThreads, 8>, dim3((unsigned)(slices * row_blocks)), dim3(kSpmmThreads), stream, nullptr, 0,
                    dev, (int)I.m, k, row_blocks, r, ranges, (const int*)p->cuts_block, p->row_ptr, col_idx, vals, B, Y, partial, alpha, beta,
                    kMediumRow);
      }
      if (partial) { const cudaError_t e = cudaFreeAsync(partial, stream); if (e != cudaSuccess && rc == B200SP_OK) rc = cuda_fail(e, "cudaFreeAsync"); }
      if (rc == B200SP_OK && p->num_medium > 0) {
        tl_pdl_kernel = true;
        rc = launch(spmm_medium_row_kernel<T, VEC, kSpmmThreads, 8>, dim3((unsigned)(slices * mid_blocks)), dim3(kSpmmThreads), stream,
                    nullptr, 0, dev, p->num_medium, (const int*)p->medium_rows, k, mid_blocks, p->row_ptr, col_idx, vals, B, Y, alpha, beta);
      }
    } else
    // rows of at most kMediumRow nonzeros: the register-capped kernel; kMediumRow + 1 .. kLongRow: the same scheme with
    // blocked sums over the plan's list of such rows; longer rows: a CTA per (row, slice)
#define B200SP_SLICE_LAUNCH(L)                                                                                                      \
    tl_pdl_kernel = true;                                                                                                           \
    if ((g_opt.spmm_stage_a == 1 || (g_opt.spmm_stage_a == 2 && sizeof(T) == 2)) && L > 1)                                          \
      rc = launch(spmm_slice_staged_kernel<T, VEC, kSpmmThreads, (L > 1 ? L : 2), kSpmmStageCap>, dim3((unsigned)(slices * row_blocks)),  \
                  dim3(kSpmmThreads), stream, B, (size_t)I.n * k * sizeof(T), dev, (int)I.m, (int)I.nnz, k, row_blocks, p->row_ptr, col_idx, vals, B, Y, alpha, \
                  beta, kMediumRow);                                                                                                \
    else                                                                                                                            \
      rc = launch(spmm_slice_kernel<T, VEC, kSpmmThreads, L>, dim3((unsigned)(slices * row_blocks)), dim3(kSpmmThreads), stream, B,       \
                  (size_t)I.n * k * sizeof(T), dev, (int)I.m, k, row_blocks, p->row_ptr, col_idx, vals, B, Y, alpha, beta, kMediumRow);                          \
    if (rc == B200SP_OK && p->num_medium > 0) {                                                                                     \
      tl_pdl_kernel = true;                                                                                                         \
      rc = launch(spmm_medium_row_kernel<T, VEC, kSpmmThreads, L>, dim3((unsigned)(slices * mid_blocks)), dim3(kSpmmThreads), stream, \
                  nullptr, 0, dev, p->num_medium, (const int*)p->medium_rows, k, mid_blocks, p->row_ptr, col_idx, vals, B, Y, alpha, beta); \
    }
    if (lanes == 8) { B200SP_SLICE_LAUNCH(8); }
    else if (lanes == 4) { B200SP_SLICE_LAUNCH(4); }
    else if (lanes == 2) { B200SP_SLICE_LAUNCH(2); }
    else { B200SP_SLICE_LAUNCH(1); }
#undef B200SP_SLICE_LAUNCH
    if (rc != B200SP_OK || p->num_long == 0) return rc;
    const long long ctas = (long long)((k + 8 * VEC - 1) / (8 * VEC)) * p->num_long;
    if (ctas >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
    tl_pdl_kernel = true;
    return launch(spmm_long_row_kernel<T, VEC, kSpmmThreads>, dim3((unsigned)ctas), dim3(kSpmmThreads), stream, nullptr, 0,
                  dev, k, p->num_long, (const int*)p->long_rows, p->row_ptr, col_idx, vals, B, Y, alpha, beta);
  }
  if (k % VEC != 0) {  // ragged k: scalar lanes
    if (k <= 2) return launch_spmm<T, 1, 2, 1>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
    if (k <= 4) return launch_spmm<T, 1, 4, 1>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
    if (k <= 8) return launch_spmm<T, 1, 8, 1>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
    return launch_spmm<T, 1, 32, 2>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  }
  const int vecs = k / VEC;  // vector columns per row
  if (vecs <= 4) return launch_spmm<T, VEC, 4, 1>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  if (vecs <= 8) return launch_spmm<T, VEC, 8, 1>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  if (vecs <= 16) return launch_spmm<T, VEC, 16, 1>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  if (vecs <= 32) return launch_spmm<T, VEC, 32, 1>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  return launch_spmm<T, VEC, 32, 2>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
}

}  // namespace
