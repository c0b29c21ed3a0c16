// Host side of libb200sp.so: the COO, CSC and ELL front ends (row offsets, transpose plan, ELL launches).
// One of the pieces of the single translation unit b200sp.cu; include/b200sp.h states the contract of every entry point.
#pragma once
#include "host_spmm.cuh"
#include "format_kernels.cuh"

// ---- COO front end: row offsets from sorted row indices, then the CSR path ----
struct CooEntry { int32_t* row_ptr = nullptr; };
static std::map<std::tuple<int, const void*, int64_t, int64_t, int64_t>, CooEntry> g_coo_cache;

static int coo_row_ptr(const int32_t** out, int64_t m, int64_t n, int64_t nnz, const int32_t* row_idx, cudaStream_t stream) {
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  int d = 0;
  CU(cudaGetDevice(&d));
  const auto key = std::make_tuple(d, (const void*)row_idx, m, n, nnz);
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    auto it = g_coo_cache.find(key);
    if (it != g_coo_cache.end()) { *out = it->second.row_ptr; return B200SP_OK; }
  }
  int32_t* rp = nullptr;
  int* d_bad = nullptr;
  int h_bad = 0;
  CU(cudaMalloc(&rp, (size_t)(m + 1) * sizeof(int32_t)));
  cudaError_t e = cudaMalloc(&d_bad, sizeof(int));
  if (e == cudaSuccess) e = cudaMemsetAsync(d_bad, 0, sizeof(int), stream);
  if (e == cudaSuccess) {
    const long long work = (m + 1 > nnz ? m + 1 : nnz);
    long long blocks = (work + 255) / 256;
    if (blocks > (long long)dev->sms * 16) blocks = (long long)dev->sms * 16;
    coo_row_ptr_kernel<<<(unsigned)blocks, 256, 0, stream>>>(row_idx, (int)nnz, (int)m, rp, d_bad);
    g_launches++;
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&h_bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (d_bad) cudaFree(d_bad);
  if (e != cudaSuccess) { cudaFree(rp); return cuda_fail(e, "COO row offsets"); }
  if (h_bad) { cudaFree(rp); return B200SP_ERR_UNSUPPORTED; }   // entries not sorted by row, or a row index out of range
  std::lock_guard<std::mutex> lock(g_mutex);
  auto ins = g_coo_cache.emplace(key, CooEntry{rp});
  if (!ins.second) { cudaFree(rp); rp = ins.first->second.row_ptr; }
  *out = rp;
  return B200SP_OK;
}

// ---- CSC front end: a transpose plan built on the device (see format_kernels.cuh), then the CSR path ----
// One pool block per pattern: row offsets, columns and CSC positions in row-major order, and room for the permuted values.
struct CscEntry { void* block = nullptr; int32_t* row_ptr = nullptr; int32_t* col = nullptr; int32_t* perm = nullptr; void* vals_t = nullptr; };
static std::map<std::tuple<int, const void*, const void*, int64_t, int64_t, int64_t>, CscEntry> g_csc_cache;

static void csc_free(CscEntry& e) {
  if (e.block) cudaFree(e.block);
  e = CscEntry();
}

static int csc_plan(CscEntry* out, int64_t m, int64_t n, int64_t nnz, const int32_t* col_ptr, const int32_t* row_idx, cudaStream_t stream) {
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  int d = 0;
  CU(cudaGetDevice(&d));
  const auto key = std::make_tuple(d, (const void*)col_ptr, (const void*)row_idx, m, n, nnz);
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    auto it = g_csc_cache.find(key);
    if (it != g_csc_cache.end()) { *out = it->second; return B200SP_OK; }
  }
  auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
  const size_t nz = nnz > 0 ? (size_t)nnz : 1;
  const size_t blocks = (size_t)((m + 1 + kScanBlock - 1) / kScanBlock);
  const size_t o_rp = 0, o_col = o_rp + up(((size_t)m + 2) * 4), o_perm = o_col + up(nz * 4), o_vals = o_perm + up(nz * 4),
               o_fill = o_vals + up(nz * 4), o_bs = o_fill + up(((size_t)m + 2) * 4), o_bad = o_bs + up((blocks + 1) * 4), total = o_bad + 256;
  CscEntry e;
  rc = pool_alloc(dev, &e.block, total, stream);
  if (rc != B200SP_OK) return rc;
  char* base = (char*)e.block;
  e.row_ptr = (int32_t*)(base + o_rp);
  e.col = (int32_t*)(base + o_col);
  e.perm = (int32_t*)(base + o_perm);
  e.vals_t = base + o_vals;
  int* fill = (int*)(base + o_fill);
  int* bsum = (int*)(base + o_bs);
  int* d_bad = (int*)(base + o_bad);
  int h_bad = 0;
  auto fail = [&](int code) { cudaFreeAsync(e.block, stream); cudaStreamSynchronize(stream); return code; };
#define CUF(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(cuda_fail(e_, #call)); } while (0)
  const unsigned wide = (unsigned)(dev->sms * 16);
  auto grid_for = [&](int64_t work) { long long b = (work + 255) / 256; if (b < 1) b = 1; return (unsigned)(b > (long long)wide ? wide : b); };
  CUF(cudaMemsetAsync(d_bad, 0, sizeof(int), stream));
  CUF(cudaMemsetAsync(fill, 0, ((size_t)m + 2) * 4, stream));
  csc_check_kernel<<<grid_for(nnz > n ? nnz : n), 256, 0, stream>>>(col_ptr, row_idx, (int)m, (int)n, (int)nnz, d_bad);
  g_launches++;
  CUF(cudaGetLastError());
  CUF(cudaMemcpyAsync(&h_bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, stream));
  CUF(cudaStreamSynchronize(stream));                          // nothing below may index with an unchecked row number
  if (h_bad) return fail(B200SP_ERR_BAD_CSR);
  if (nnz > 0) csc_count_rows_kernel<<<grid_for(nnz), 256, 0, stream>>>(row_idx, (long long)nnz, fill);
  // exclusive scan of the m + 1 counts (the last one is zero) -> row offsets, row_ptr[m] = nnz
  scan_block_sums_kernel<<<(unsigned)blocks, 256, 0, stream>>>(fill, (long long)m + 1, bsum);
  plan_compact_scan_kernel<<<1, 1024, 0, stream>>>(bsum, (int)blocks);
  scan_apply_kernel<<<(unsigned)blocks, 256, 0, stream>>>(fill, (long long)m + 1, bsum, e.row_ptr);
  g_launches += 4;
  CUF(cudaGetLastError());
  CUF(cudaMemsetAsync(fill, 0, ((size_t)m + 2) * 4, stream));
  if (nnz > 0) {
    csc_place_kernel<<<grid_for(nnz), 256, 0, stream>>>(row_idx, (long long)nnz, e.row_ptr, fill, e.perm);
    csc_sort_rows_kernel<<<(unsigned)((m + 255) / 256), 256, 0, stream>>>((int)m, e.row_ptr, e.perm);
    csc_cols_kernel<<<grid_for(nnz), 256, 0, stream>>>((long long)nnz, (int)n, col_ptr, e.perm, e.col);
    g_launches += 3;
    CUF(cudaGetLastError());
  }
  CUF(cudaStreamSynchronize(stream));
#undef CUF
  std::lock_guard<std::mutex> lock(g_mutex);
  auto ins = g_csc_cache.emplace(key, e);
  if (!ins.second) { cudaFreeAsync(e.block, stream); e = ins.first->second; }
  *out = e;
  return B200SP_OK;
}

static int csc_call(bool is_mm, int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* col_ptr, const int32_t* row_idx, const void* vals,
                    const void* in, void* out, float alpha, float beta, int dtype, void* stream_v) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (k <= 0) return B200SP_ERR_INVALID_ARG;
  if (!col_ptr || (nnz > 0 && (!row_idx || !vals))) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  cudaStream_t stream = (cudaStream_t)stream_v;
  CscEntry e;
  rc = csc_plan(&e, m, n, nnz, col_ptr, row_idx, stream);
  if (rc != B200SP_OK) return rc;
  if (nnz > 0) {
    long long blocks = (nnz + 255) / 256;
    if (blocks > (long long)dev->sms * 16) blocks = (long long)dev->sms * 16;
    rc = dtype == B200SP_F32
             ? launch(csc_permute_vals_kernel<float>, dim3((unsigned)blocks), dim3(256), stream, nullptr, 0, dev, (long long)nnz, (const int*)e.perm, (const float*)vals, (float*)e.vals_t)
             : launch(csc_permute_vals_kernel<bf16_t>, dim3((unsigned)blocks), dim3(256), stream, nullptr, 0, dev, (long long)nnz, (const int*)e.perm, (const bf16_t*)vals, (bf16_t*)e.vals_t);
    if (rc != B200SP_OK) return rc;
  }
  return is_mm ? spmm_csr(m, n, nnz, k, e.row_ptr, e.col, e.vals_t, in, out, alpha, beta, dtype, stream_v)
               : spmv_csr(m, n, nnz, e.row_ptr, e.col, e.vals_t, in, out, alpha, beta, dtype, stream_v);
}

// ---- ELL front end ----
static int check_ell(int64_t m, int64_t n, int64_t width, const void* col_ids, const void* vals, const void* in, const void* out, int dtype) {
  if (m < 0 || n < 0 || width < 0 || n >= ((int64_t)1 << 31) || m >= ((int64_t)1 << 31) - 1) return B200SP_ERR_INVALID_ARG;
  if (m * width >= ((int64_t)1 << 31)) return B200SP_ERR_INVALID_ARG;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (m > 0 && !out) return B200SP_ERR_INVALID_ARG;
  if (m * width > 0 && (!col_ids || !vals || !in)) return B200SP_ERR_INVALID_ARG;
  if (!aligned16(col_ids) || !aligned16(vals) || !aligned16(in) || !aligned16(out)) return B200SP_ERR_INVALID_ARG;
  return B200SP_OK;
}

template <typename T, int LPR, int VECW>
static int launch_ell_spmv(int64_t m, int width, const int32_t* col_ids, const T* vals, const T* x, T* y, float alpha, float beta,
                           cudaStream_t stream, DeviceInfo* dev) {
  constexpr int THREADS = 128;
  const long long blocks = (m * LPR + THREADS - 1) / THREADS;
  if (blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  tl_pdl_kernel = true;
  return launch(spmv_ell_kernel<T, LPR, VECW, THREADS>, dim3((unsigned)blocks), dim3(THREADS), stream, nullptr, 0, dev, (int)m, width, col_ids,
                vals, x, y, alpha, beta);
}

template <typename T>
static int run_ell_spmv(int64_t m, int width, const int32_t* col_ids, const T* vals, const T* x, T* y, float alpha, float beta,
                        cudaStream_t stream, DeviceInfo* dev) {
  if (m == 0) return B200SP_OK;
  if (alpha == 0.0f || width == 0) return run_scale<T>(m, y, beta, stream, dev);
  if (width % 4 != 0 && width <= kRowMaxLen)   // odd widths (stencils): the staged row-direct kernel with implicit row offsets
    return launch_row_direct_ell<T>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
  if (width % 4 == 0) {   // 128-bit loads: lanes per row = largest power of two not above width / 4 (at most 32)
    const int q = width / 4;
    if (q >= 32) return launch_ell_spmv<T, 32, 4>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
    if (q >= 16) return launch_ell_spmv<T, 16, 4>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
    if (q >= 8) return launch_ell_spmv<T, 8, 4>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
    if (q >= 4) return launch_ell_spmv<T, 4, 4>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
    if (q >= 2) return launch_ell_spmv<T, 2, 4>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
    return launch_ell_spmv<T, 1, 4>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
  }
  if (width >= 32) return launch_ell_spmv<T, 16, 1>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
  if (width >= 12) return launch_ell_spmv<T, 8, 1>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
  if (width >= 6) return launch_ell_spmv<T, 4, 1>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
  if (width >= 3) return launch_ell_spmv<T, 2, 1>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
  return launch_ell_spmv<T, 1, 1>(m, width, col_ids, vals, x, y, alpha, beta, stream, dev);
}

template <typename T, int VEC>
static int run_ell_spmm(int64_t m, int width, int k, const int32_t* col_ids, const T* vals, const T* B, T* Y, float alpha, float beta,
                        cudaStream_t stream, DeviceInfo* dev) {
  if (m == 0) return B200SP_OK;
  if (alpha == 0.0f || width == 0) return run_scale<T>((long long)m * k, Y, beta, stream, dev);
  if (k % VEC == 0) {
    constexpr int KS = 8 * VEC, GROUPS = kSpmmThreads / 8;
    const int slices = (k + KS - 1) / KS;
    const int row_blocks = (int)((m + GROUPS - 1) / GROUPS);
    if ((long long)slices * row_blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
    return launch(spmm_ell_slice_kernel<T, VEC, kSpmmThreads>, dim3((unsigned)(slices * row_blocks)), dim3(kSpmmThreads), stream, nullptr, 0, dev,
                  (int)m, k, width, row_blocks, col_ids, vals, B, Y, alpha, beta);
  }
  const long long blocks = ((long long)m * k + 255) / 256;
  if (blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  return launch(spmm_ell_entry_kernel<T>, dim3((unsigned)blocks), dim3(256), stream, nullptr, 0, dev, (long long)m, k, width, col_ids, vals, B, Y,
                alpha, beta);
}

