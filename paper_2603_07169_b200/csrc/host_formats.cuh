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

// ---- CSC front end: a transpose plan (built on the host, stable in column order), then the CSR path ----
struct CscEntry { int32_t* row_ptr = nullptr; int32_t* col = nullptr; int32_t* perm = nullptr; void* vals_t = nullptr; };
static std::map<std::tuple<int, const void*, const void*, int64_t, int64_t, int64_t>, CscEntry> g_csc_cache;

static void csc_free(CscEntry& e) {
  for (void* q : {(void*)e.row_ptr, (void*)e.col, (void*)e.perm, e.vals_t}) if (q) cudaFree(q);
  e = CscEntry();
}

static int csc_plan(CscEntry* out, int64_t m, int64_t n, int64_t nnz, const int32_t* col_ptr, const int32_t* row_idx, cudaStream_t stream) {
  int d = 0;
  CU(cudaGetDevice(&d));
  const auto key = std::make_tuple(d, (const void*)col_ptr, (const void*)row_idx, m, n, nnz);
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    auto it = g_csc_cache.find(key);
    if (it != g_csc_cache.end()) { *out = it->second; return B200SP_OK; }
  }
  // pattern to the host, stable counting sort by row (entries of a row end up in ascending column order), back to the device
  std::vector<int32_t> h_cp((size_t)n + 1), h_ri((size_t)nnz), h_rp((size_t)m + 1, 0), h_col((size_t)nnz), h_perm((size_t)nnz);
  CU(cudaMemcpyAsync(h_cp.data(), col_ptr, ((size_t)n + 1) * 4, cudaMemcpyDeviceToHost, stream));
  if (nnz > 0) CU(cudaMemcpyAsync(h_ri.data(), row_idx, (size_t)nnz * 4, cudaMemcpyDeviceToHost, stream));
  CU(cudaStreamSynchronize(stream));
  if (h_cp[0] != 0 || h_cp[(size_t)n] != nnz) return B200SP_ERR_BAD_CSR;
  for (int64_t p = 0; p < nnz; ++p) {
    if (h_ri[(size_t)p] < 0 || h_ri[(size_t)p] >= m) return B200SP_ERR_BAD_CSR;
    h_rp[(size_t)h_ri[(size_t)p] + 1]++;
  }
  for (int64_t i = 0; i < m; ++i) h_rp[(size_t)i + 1] += h_rp[(size_t)i];
  {
    std::vector<int32_t> next(h_rp.begin(), h_rp.end() - 1);
    for (int64_t j = 0; j < n; ++j) {
      if (h_cp[(size_t)j + 1] < h_cp[(size_t)j]) return B200SP_ERR_BAD_CSR;
      for (int32_t p = h_cp[(size_t)j]; p < h_cp[(size_t)j + 1]; ++p) {
        const int32_t q = next[(size_t)h_ri[(size_t)p]]++;
        h_col[(size_t)q] = (int32_t)j;
        h_perm[(size_t)q] = p;
      }
    }
  }
  CscEntry e;
  auto fail = [&](cudaError_t err, const char* what) { csc_free(e); return cuda_fail(err, what); };
  cudaError_t err;
  if ((err = cudaMalloc(&e.row_ptr, ((size_t)m + 1) * 4)) != cudaSuccess) return fail(err, "cudaMalloc");
  const size_t nz = nnz > 0 ? (size_t)nnz : 1;
  if ((err = cudaMalloc(&e.col, nz * 4)) != cudaSuccess) return fail(err, "cudaMalloc");
  if ((err = cudaMalloc(&e.perm, nz * 4)) != cudaSuccess) return fail(err, "cudaMalloc");
  if ((err = cudaMalloc(&e.vals_t, nz * 4)) != cudaSuccess) return fail(err, "cudaMalloc");
  if ((err = cudaMemcpyAsync(e.row_ptr, h_rp.data(), ((size_t)m + 1) * 4, cudaMemcpyHostToDevice, stream)) != cudaSuccess) return fail(err, "cudaMemcpyAsync");
  if (nnz > 0) {
    if ((err = cudaMemcpyAsync(e.col, h_col.data(), (size_t)nnz * 4, cudaMemcpyHostToDevice, stream)) != cudaSuccess) return fail(err, "cudaMemcpyAsync");
    if ((err = cudaMemcpyAsync(e.perm, h_perm.data(), (size_t)nnz * 4, cudaMemcpyHostToDevice, stream)) != cudaSuccess) return fail(err, "cudaMemcpyAsync");
  }
  if ((err = cudaStreamSynchronize(stream)) != cudaSuccess) return fail(err, "cudaStreamSynchronize");
  std::lock_guard<std::mutex> lock(g_mutex);
  auto ins = g_csc_cache.emplace(key, e);
  if (!ins.second) { csc_free(e); e = ins.first->second; }
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

