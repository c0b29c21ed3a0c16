// C ABI of libb200sp.so: argument checks, plan pass, kernel selection and launches.
// The operations are those of the paper's Appendix C, Table 6, tasks 12 (SpMV CSR) and 13 (SpMM CSR),
// generalised with alpha / beta; see include/b200sp.h for the contract of every entry point.
// The host code is split by topic over host_runtime / host_plan / host_spmv / host_spmm / host_formats (.cuh); this file
// holds the extern "C" entry points.
#include "host_formats.cuh"

// ---- scratch for spmv_csr_noalloc: lives in the library image, one copy per GPU that loads it ----
constexpr int kNoAllocMaxTiles = 65536;   // merge tiles of kItems items: m + nnz <= 65536 * 4096 = 268,435,456
struct NoAllocScratch {
  int32_t split_row[kNoAllocMaxTiles + 4];
  float carry[kNoAllocMaxTiles];
  float tail[kNoAllocMaxTiles];
};
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];
// In host code the name above is only a handle; the device address comes from cudaGetSymbolAddress,
// looked up once per device with that device current.
static NoAllocScratch* g_noalloc_ptr[64] = {};

static int noalloc_scratch(NoAllocScratch** out) {
  int dev = 0;
  CU(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return B200SP_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_noalloc_ptr[dev]) {
    void* ptr = nullptr;
    CU(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
    g_noalloc_ptr[dev] = static_cast<NoAllocScratch*>(ptr);
  }
  *out = g_noalloc_ptr[dev];
  return B200SP_OK;
}

template <typename T>
static int run_spmv_noalloc(int64_t m, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, const T* vals, const T* x, T* y,
                            float alpha, float beta, cudaStream_t stream, DeviceInfo* dev, NoAllocScratch* sc) {
  if (alpha == 0.0f || nnz == 0) return run_scale<T>(m, y, beta, stream, dev);
  const int tiles = (int)((m + nnz + kItems - 1) / kItems);
  int rc = launch(plan_merge_split_kernel, dim3((tiles + 1 + 255) / 256), dim3(256), stream, nullptr, 0, dev, row_ptr, (int)m, (int)nnz,
                  kItems, tiles, (int*)sc->split_row);
  if (rc != B200SP_OK) return rc;
  rc = launch(spmv_merge_tile_kernel<T, kItems, kThreads, kShortMax>, dim3(tiles), dim3(kThreads), stream, nullptr, 0, dev, (int)m,
              (int)nnz, row_ptr, col_idx, vals, x, y, alpha, beta, (const int*)sc->split_row, sc->carry, sc->tail, (const int*)nullptr);
  if (rc != B200SP_OK) return rc;
  if (tiles > 1)
    rc = launch(spmv_carry_fixup_kernel<T, kItems>, dim3((tiles + 127) / 128), dim3(128), stream, nullptr, 0, dev, tiles, row_ptr,
                (const int*)sc->split_row, (const float*)sc->carry, (const float*)sc->tail, y, alpha, beta, (const int*)nullptr);
  return rc;
}

// ---- checked build (-DB200SP_BOUNDS_CHECK): every compute call first verifies on the device that row_ptr is monotone
// with the right ends and that every column index lies in [0, n), synchronises, and refuses an inconsistent matrix with
// B200SP_ERR_BAD_CSR before any kernel that would index with it is launched.  A stand-in for a memory checker: nothing
// traps, the first bad matrix is reported by a status code.  The ordinary build compiles this away.
static int checked_build_validate(const b200sp_plan* p, const int32_t* col_idx, void* stream) {
#ifdef B200SP_BOUNDS_CHECK
  const b200sp_plan_info_t& I = p->info;
  if (I.m == 0) return B200SP_OK;
  return b200sp_validate_csr(I.m, I.n, I.nnz, p->row_ptr, col_idx, stream);
#else
  (void)p; (void)col_idx; (void)stream;
  return B200SP_OK;
#endif
}

// launcher of the gather probe (b200sp_tuning.h)
template <typename E, bool SMEM>
static int run_probe_gather(const void* table, int64_t table_elems, int64_t gathers, float* sink, cudaStream_t stream, DeviceInfo* dev) {
  auto kernel = probe_gather_kernel<E, SMEM>;
  const size_t smem = SMEM ? (size_t)table_elems * sizeof(E) : 0;
  int d = 0;
  CU(cudaGetDevice(&d));
  if (SMEM) {
    if (smem > (size_t)kSmemPerSm - 2048) return B200SP_ERR_INVALID_ARG;
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  } else {
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 0));
  }
  int nb = 0;
  CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kernel, 256, smem));
  if (nb < 1) nb = 1;
  return launch_smem(kernel, dim3((unsigned)(dev->sms * nb)), dim3(256), smem, stream, nullptr, 0, dev, (const E*)table,
                     (unsigned)(table_elems - 1), (long long)gathers, sink);
}

extern "C" {

int b200sp_plan_create(b200sp_plan** out, int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, void* stream) {
  if (!out) return B200SP_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (m > 0 && (!row_ptr || !aligned4(row_ptr))) return B200SP_ERR_INVALID_ARG;
  return plan_build(out, m, n, nnz, row_ptr, (cudaStream_t)stream);
}

int b200sp_plan_destroy(b200sp_plan* plan) { return plan_free(plan); }

int b200sp_plan_info(const b200sp_plan* plan, b200sp_plan_info_t* out) {
  if (!plan || !out) return B200SP_ERR_INVALID_ARG;
  *out = plan->info;
  return B200SP_OK;
}

int b200sp_spmv(b200sp_plan* plan, const int32_t* col_idx, const void* vals, const void* x, void* y, float alpha, float beta,
                int dtype, void* stream) {
  int rc = check_common(plan, col_idx, vals, x, y, dtype);
  if (rc != B200SP_OK) return rc;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  rc = checked_build_validate(plan, col_idx, stream);
  if (rc != B200SP_OK) return rc;
  if (dtype == B200SP_F32) return run_spmv<float>(plan, col_idx, (const float*)vals, (const float*)x, (float*)y, alpha, beta, (cudaStream_t)stream, dev);
  return run_spmv<bf16_t>(plan, col_idx, (const bf16_t*)vals, (const bf16_t*)x, (bf16_t*)y, alpha, beta, (cudaStream_t)stream, dev);
}

int b200sp_spmm(b200sp_plan* plan, int64_t k, const int32_t* col_idx, const void* vals, const void* B, void* Y, float alpha,
                float beta, int dtype, void* stream) {
  int rc = check_common(plan, col_idx, vals, B, Y, dtype);
  if (rc != B200SP_OK) return rc;
  if (k <= 0 || k >= ((int64_t)1 << 31) || plan->info.m * k >= ((int64_t)1 << 40)) return B200SP_ERR_INVALID_ARG;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  rc = checked_build_validate(plan, col_idx, stream);
  if (rc != B200SP_OK) return rc;
  if (dtype == B200SP_F32) return run_spmm<float, 4>(plan, (int)k, col_idx, (const float*)vals, (const float*)B, (float*)Y, alpha, beta, (cudaStream_t)stream, dev);
  return run_spmm<bf16_t, 8>(plan, (int)k, col_idx, (const bf16_t*)vals, (const bf16_t*)B, (bf16_t*)Y, alpha, beta, (cudaStream_t)stream, dev);
}

int spmv_csr(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, const void* vals, const void* x,
             void* y, float alpha, float beta, int dtype, void* stream) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (m > 0 && (!row_ptr || !y)) return B200SP_ERR_INVALID_ARG;
  if (nnz > 0 && (!col_idx || !vals || !x)) return B200SP_ERR_INVALID_ARG;
  if (!aligned4(row_ptr) || !aligned16(col_idx) || !aligned16(vals) || !aligned16(x) || !aligned16(y)) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  b200sp_plan* p = nullptr;
  rc = get_cached_plan(&p, m, n, nnz, row_ptr, (cudaStream_t)stream);
  if (rc != B200SP_OK) return rc;
  return b200sp_spmv(p, col_idx, vals, x, y, alpha, beta, dtype, stream);
}

int spmm_csr(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr, const int32_t* col_idx, const void* vals,
             const void* B, void* Y, float alpha, float beta, int dtype, void* stream) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (k <= 0) return B200SP_ERR_INVALID_ARG;
  if (m > 0 && (!row_ptr || !Y)) return B200SP_ERR_INVALID_ARG;
  if (nnz > 0 && (!col_idx || !vals || !B)) return B200SP_ERR_INVALID_ARG;
  if (!aligned4(row_ptr) || !aligned16(col_idx) || !aligned16(vals) || !aligned16(B) || !aligned16(Y)) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  b200sp_plan* p = nullptr;
  rc = get_cached_plan(&p, m, n, nnz, row_ptr, (cudaStream_t)stream);
  if (rc != B200SP_OK) return rc;
  return b200sp_spmm(p, k, col_idx, vals, B, Y, alpha, beta, dtype, stream);
}

int spmv_csr_noalloc(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, const void* vals,
                     const void* x, void* y, float alpha, float beta, int dtype, void* stream) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (m > 0 && (!row_ptr || !y)) return B200SP_ERR_INVALID_ARG;
  if (nnz > 0 && (!col_idx || !vals || !x)) return B200SP_ERR_INVALID_ARG;
  if (!aligned4(row_ptr) || !aligned16(col_idx) || !aligned16(vals) || !aligned16(x) || !aligned16(y)) return B200SP_ERR_INVALID_ARG;
  if (m + nnz > (int64_t)kNoAllocMaxTiles * kItems) return B200SP_ERR_TOO_LARGE;   // beyond the built-in scratch
  if (m == 0) return B200SP_OK;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  NoAllocScratch* sc = nullptr;
  rc = noalloc_scratch(&sc);
  if (rc != B200SP_OK) return rc;
  if (dtype == B200SP_F32)
    return run_spmv_noalloc<float>(m, nnz, row_ptr, col_idx, (const float*)vals, (const float*)x, (float*)y, alpha, beta, (cudaStream_t)stream, dev, sc);
  return run_spmv_noalloc<bf16_t>(m, nnz, row_ptr, col_idx, (const bf16_t*)vals, (const bf16_t*)x, (bf16_t*)y, alpha, beta, (cudaStream_t)stream, dev, sc);
}

int b200sp_spmv_naive(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, const void* vals,
                      const void* x, void* y, float alpha, float beta, int dtype, void* stream) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (m > 0 && (!row_ptr || !y)) return B200SP_ERR_INVALID_ARG;
  if (nnz > 0 && (!col_idx || !vals || !x)) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  const unsigned blocks = (unsigned)((m + 255) / 256);
  if (dtype == B200SP_F32)
    return launch(spmv_naive_kernel<float>, dim3(blocks), dim3(256), (cudaStream_t)stream, nullptr, 0, dev, (int)m, row_ptr, col_idx,
                  (const float*)vals, (const float*)x, (float*)y, alpha, beta);
  return launch(spmv_naive_kernel<bf16_t>, dim3(blocks), dim3(256), (cudaStream_t)stream, nullptr, 0, dev, (int)m, row_ptr, col_idx,
                (const bf16_t*)vals, (const bf16_t*)x, (bf16_t*)y, alpha, beta);
}

int b200sp_spmm_naive(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr, const int32_t* col_idx, const void* vals,
                      const void* B, void* Y, float alpha, float beta, int dtype, void* stream) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (k <= 0 || k >= ((int64_t)1 << 31)) return B200SP_ERR_INVALID_ARG;
  if (m > 0 && (!row_ptr || !Y)) return B200SP_ERR_INVALID_ARG;
  if (nnz > 0 && (!col_idx || !vals || !B)) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  const long long blocks = (m * k + 255) / 256;
  if (blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  if (dtype == B200SP_F32)
    return launch(spmm_naive_kernel<float>, dim3((unsigned)blocks), dim3(256), (cudaStream_t)stream, nullptr, 0, dev, (long long)m, (int)k,
                  row_ptr, col_idx, (const float*)vals, (const float*)B, (float*)Y, alpha, beta);
  return launch(spmm_naive_kernel<bf16_t>, dim3((unsigned)blocks), dim3(256), (cudaStream_t)stream, nullptr, 0, dev, (long long)m, (int)k,
                row_ptr, col_idx, (const bf16_t*)vals, (const bf16_t*)B, (bf16_t*)Y, alpha, beta);
}

// ---- measurement probes (b200sp_tuning.h) ----
int b200sp_probe_gather_ex(const void* table, int64_t table_elems, int64_t gathers, int elem_bytes, int in_shared_memory, float* sink,
                           void* stream) {
  if (!table || !sink || table_elems <= 0 || (table_elems & (table_elems - 1)) != 0 || table_elems > ((int64_t)1 << 31) || gathers < 0 ||
      (elem_bytes != 2 && elem_bytes != 4))
    return B200SP_ERR_INVALID_ARG;
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (elem_bytes == 4)
    return in_shared_memory ? run_probe_gather<float, true>(table, table_elems, gathers, sink, st, dev)
                            : run_probe_gather<float, false>(table, table_elems, gathers, sink, st, dev);
  return in_shared_memory ? run_probe_gather<unsigned short, true>(table, table_elems, gathers, sink, st, dev)
                          : run_probe_gather<unsigned short, false>(table, table_elems, gathers, sink, st, dev);
}

int b200sp_probe_gather(const float* table, int64_t table_elems, int64_t gathers, float* sink, void* stream) {
  return b200sp_probe_gather_ex(table, table_elems, gathers, 4, 0, sink, stream);
}

int b200sp_probe_stream(const void* buf, int64_t bytes, float* sink, void* stream) {
  if (!buf || !sink || bytes < 0 || (bytes & 15) || !aligned16(buf)) return B200SP_ERR_INVALID_ARG;
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  return launch(probe_stream_kernel, dim3((unsigned)(dev->sms * 8)), dim3(256), (cudaStream_t)stream, nullptr, 0, dev, (const int4*)buf,
                (long long)(bytes / 16), sink);
}

int b200sp_probe_lines(const void* buf, int64_t lines, int64_t reads, int in_flight, int to_shared_memory, int group_lanes, float* sink,
                       void* stream) {
  if (!buf || !sink || lines <= 0 || (lines & (lines - 1)) != 0 || lines > ((int64_t)1 << 31) || reads < 0 || !aligned16(buf) ||
      (in_flight != 4 && in_flight != 8 && in_flight != 16) || (group_lanes != 8 && group_lanes != 16 && group_lanes != 32) ||
      lines < group_lanes / 8 || (to_shared_memory && group_lanes != 8))
    return B200SP_ERR_INVALID_ARG;
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const dim3 grid((unsigned)(dev->sms * 8)), block(256);
  const unsigned mask = (unsigned)(lines / (group_lanes / 8) - 1);      // chunks of group_lanes / 8 lines
  const size_t smem = to_shared_memory ? (size_t)256 * in_flight * 16 : 0;
#define B200SP_PROBE_LINES(U, A, GL) return launch_smem(probe_lines_kernel<U, A, GL>, grid, block, smem, st, nullptr, 0, dev, (const int4*)buf, mask, (long long)reads, sink)
  if (to_shared_memory) {
    if (in_flight == 4) B200SP_PROBE_LINES(4, true, 8);
    if (in_flight == 8) B200SP_PROBE_LINES(8, true, 8);
    CU(cudaFuncSetAttribute(probe_lines_kernel<16, true, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    B200SP_PROBE_LINES(16, true, 8);
  }
  if (group_lanes == 16) { if (in_flight == 4) B200SP_PROBE_LINES(4, false, 16); if (in_flight == 8) B200SP_PROBE_LINES(8, false, 16); B200SP_PROBE_LINES(16, false, 16); }
  if (group_lanes == 32) { if (in_flight == 4) B200SP_PROBE_LINES(4, false, 32); if (in_flight == 8) B200SP_PROBE_LINES(8, false, 32); B200SP_PROBE_LINES(16, false, 32); }
  if (in_flight == 4) B200SP_PROBE_LINES(4, false, 8);
  if (in_flight == 8) B200SP_PROBE_LINES(8, false, 8);
  B200SP_PROBE_LINES(16, false, 8);
#undef B200SP_PROBE_LINES
}

int b200sp_probe_spmv_gather(int64_t nnz, const int32_t* col_idx, const void* vals, const void* x, int dtype, int unused_smem_kb, float* out,
                             void* stream) {
  if (!col_idx || !vals || !x || !out || nnz < 4 || nnz >= ((int64_t)1 << 31) || !aligned16(col_idx) || !aligned16(vals) ||
      (dtype != B200SP_F32 && dtype != B200SP_BF16) || unused_smem_kb < 0 || unused_smem_kb > 200)
    return B200SP_ERR_INVALID_ARG;
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  const size_t smem = (size_t)unused_smem_kb * 1024;
  const dim3 grid((unsigned)dev->sms), block(1024);
  if (dtype == B200SP_F32) {
    CU(cudaFuncSetAttribute(probe_spmv_gather_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    return launch_smem(probe_spmv_gather_kernel<float>, grid, block, smem, (cudaStream_t)stream, nullptr, 0, dev, (const int*)col_idx,
                       (const float*)vals, (long long)(nnz / 4), (const float*)x, out);
  }
  CU(cudaFuncSetAttribute(probe_spmv_gather_kernel<bf16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
  return launch_smem(probe_spmv_gather_kernel<bf16_t>, grid, block, smem, (cudaStream_t)stream, nullptr, 0, dev, (const int*)col_idx,
                     (const bf16_t*)vals, (long long)(nnz / 4), (const bf16_t*)x, out);
}

int64_t b200sp_noalloc_max_items(void) { return (int64_t)kNoAllocMaxTiles * kItems; }

int spmv_coo(int64_t m, int64_t n, int64_t nnz, const int32_t* row_idx, const int32_t* col_idx, const void* vals, const void* x,
             void* y, float alpha, float beta, int dtype, void* stream) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (nnz > 0 && !row_idx) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  const int32_t* rp = nullptr;
  rc = coo_row_ptr(&rp, m, n, nnz, row_idx, (cudaStream_t)stream);
  if (rc != B200SP_OK) return rc;
  return spmv_csr(m, n, nnz, rp, col_idx, vals, x, y, alpha, beta, dtype, stream);
}

int spmm_coo(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_idx, const int32_t* col_idx, const void* vals,
             const void* B, void* Y, float alpha, float beta, int dtype, void* stream) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (nnz > 0 && !row_idx) return B200SP_ERR_INVALID_ARG;
  if (k <= 0) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  const int32_t* rp = nullptr;
  rc = coo_row_ptr(&rp, m, n, nnz, row_idx, (cudaStream_t)stream);
  if (rc != B200SP_OK) return rc;
  return spmm_csr(m, n, nnz, k, rp, col_idx, vals, B, Y, alpha, beta, dtype, stream);
}

int spmv_csc(int64_t m, int64_t n, int64_t nnz, const int32_t* col_ptr, const int32_t* row_idx, const void* vals, const void* x, void* y,
             float alpha, float beta, int dtype, void* stream) {
  return csc_call(false, m, n, nnz, 1, col_ptr, row_idx, vals, x, y, alpha, beta, dtype, stream);
}
int spmm_csc(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* col_ptr, const int32_t* row_idx, const void* vals, const void* B,
             void* Y, float alpha, float beta, int dtype, void* stream) {
  return csc_call(true, m, n, nnz, k, col_ptr, row_idx, vals, B, Y, alpha, beta, dtype, stream);
}

int spmv_ell(int64_t m, int64_t n, int64_t width, const int32_t* col_ids, const void* vals, const void* x, void* y, float alpha, float beta,
             int dtype, void* stream) {
  int rc = check_ell(m, n, width, col_ids, vals, x, y, dtype);
  if (rc != B200SP_OK) return rc;
  if (m == 0) return B200SP_OK;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  if (dtype == B200SP_F32) return run_ell_spmv<float>(m, (int)width, col_ids, (const float*)vals, (const float*)x, (float*)y, alpha, beta, (cudaStream_t)stream, dev);
  return run_ell_spmv<bf16_t>(m, (int)width, col_ids, (const bf16_t*)vals, (const bf16_t*)x, (bf16_t*)y, alpha, beta, (cudaStream_t)stream, dev);
}

int spmm_ell(int64_t m, int64_t n, int64_t width, int64_t k, const int32_t* col_ids, const void* vals, const void* B, void* Y, float alpha,
             float beta, int dtype, void* stream) {
  int rc = check_ell(m, n, width, col_ids, vals, B, Y, dtype);
  if (rc != B200SP_OK) return rc;
  if (k <= 0 || k >= ((int64_t)1 << 31) || m * k >= ((int64_t)1 << 40)) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  if (dtype == B200SP_F32)
    return run_ell_spmm<float, 4>(m, (int)width, (int)k, col_ids, (const float*)vals, (const float*)B, (float*)Y, alpha, beta, (cudaStream_t)stream, dev);
  return run_ell_spmm<bf16_t, 8>(m, (int)width, (int)k, col_ids, (const bf16_t*)vals, (const bf16_t*)B, (bf16_t*)Y, alpha, beta, (cudaStream_t)stream, dev);
}

// ---- host-buffer entry points: copy in, plan, run, copy out, synchronise ----
static int host_call(bool is_mm, int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr, const int32_t* col_idx,
                     const void* vals, const void* in, void* out, float alpha, float beta, int dtype, void* stream_v) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (k <= 0) return B200SP_ERR_INVALID_ARG;
  if (m > 0 && (!row_ptr || !out)) return B200SP_ERR_INVALID_ARG;
  if (nnz > 0 && (!col_idx || !vals || !in)) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  cudaStream_t stream = (cudaStream_t)stream_v;
  const size_t e = dtype == B200SP_F32 ? 4 : 2;
  const size_t b_rp = (size_t)(m + 1) * 4, b_ci = (size_t)nnz * 4, b_va = (size_t)nnz * e, b_in = (size_t)n * k * e, b_out = (size_t)m * k * e;
  auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
  const size_t total = up(b_rp) + up(b_ci) + up(b_va) + up(b_in) + up(b_out) + 256;
  char* base = nullptr;
  rc = pool_alloc(dev, (void**)&base, total, stream);
  if (rc != B200SP_OK) return rc;
  char* d_rp = base; char* d_ci = d_rp + up(b_rp); char* d_va = d_ci + up(b_ci); char* d_in = d_va + up(b_va); char* d_out = d_in + up(b_in);
  // the plan is cached under the HOST address of row_ptr: a later call with the same address and sizes skips the plan pass
  // (the header states that the contents must then be unchanged, as for the device entry points)
  int cur_dev = 0;
  CU(cudaGetDevice(&cur_dev));
  const PlanKey key = std::make_tuple(cur_dev, (const void*)row_ptr, m, n, nnz);
  b200sp_plan* p = cache_find(key);
  auto done = [&](int code) { cudaFreeAsync(base, stream); cudaStreamSynchronize(stream); return code; };
#define CUH(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return done(cuda_fail(e_, #call)); } while (0)
  CUH(cudaMemcpyAsync(d_rp, row_ptr, b_rp, cudaMemcpyHostToDevice, stream));
  if (nnz > 0) {
    CUH(cudaMemcpyAsync(d_ci, col_idx, b_ci, cudaMemcpyHostToDevice, stream));
    CUH(cudaMemcpyAsync(d_va, vals, b_va, cudaMemcpyHostToDevice, stream));
    CUH(cudaMemcpyAsync(d_in, in, b_in, cudaMemcpyHostToDevice, stream));
  }
  if (beta != 0.0f) CUH(cudaMemcpyAsync(d_out, out, b_out, cudaMemcpyHostToDevice, stream));
  if (!p) {
    rc = plan_build(&p, m, n, nnz, (const int32_t*)d_rp, stream);
    if (rc != B200SP_OK) return done(rc);
    p = cache_insert(key, p);
  }
  p->row_ptr = (const int32_t*)d_rp;             // this call's staging copy
  if (p->probed_key == (const void*)col_idx) p->probed_col_idx = d_ci;   // the column-locality verdict follows the host pattern
  else p->probed_col_idx = nullptr;
  rc = is_mm ? b200sp_spmm(p, k, (const int32_t*)d_ci, d_va, d_in, d_out, alpha, beta, dtype, stream)
             : b200sp_spmv(p, (const int32_t*)d_ci, d_va, d_in, d_out, alpha, beta, dtype, stream);
  if (rc != B200SP_OK) return done(rc);
  if (p->probed_col_idx == (const void*)d_ci) p->probed_key = col_idx;
  CUH(cudaMemcpyAsync(out, d_out, b_out, cudaMemcpyDeviceToHost, stream));
  CUH(cudaStreamSynchronize(stream));
#undef CUH
  return done(B200SP_OK);
}

// Matrix resident on the device, vectors on the host (the shape of an iterative solver's step).
int spmv_csr_vec_host(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, const void* vals, const void* x_host,
                      void* y_host, float alpha, float beta, int dtype, void* stream_v) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  if (m > 0 && (!row_ptr || !y_host)) return B200SP_ERR_INVALID_ARG;
  if (nnz > 0 && (!col_idx || !vals || !x_host)) return B200SP_ERR_INVALID_ARG;
  if (m == 0) return B200SP_OK;
  cudaStream_t stream = (cudaStream_t)stream_v;
  const size_t e = dtype == B200SP_F32 ? 4 : 2;
  const size_t bx = ((size_t)n * e + 255) & ~(size_t)255, by = (size_t)m * e;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  char* base = nullptr;
  rc = pool_alloc(dev, (void**)&base, bx + by + 256, stream);
  if (rc != B200SP_OK) return rc;
  auto done = [&](int code) { cudaFreeAsync(base, stream); cudaStreamSynchronize(stream); return code; };
  cudaError_t err = cudaSuccess;
  if (n > 0) err = cudaMemcpyAsync(base, x_host, (size_t)n * e, cudaMemcpyHostToDevice, stream);
  if (err == cudaSuccess && beta != 0.0f) err = cudaMemcpyAsync(base + bx, y_host, by, cudaMemcpyHostToDevice, stream);
  if (err != cudaSuccess) return done(cuda_fail(err, "cudaMemcpyAsync"));
  rc = spmv_csr(m, n, nnz, row_ptr, col_idx, vals, base, base + bx, alpha, beta, dtype, stream_v);
  if (rc != B200SP_OK) return done(rc);
  err = cudaMemcpyAsync(y_host, base + bx, by, cudaMemcpyDeviceToHost, stream);
  if (err == cudaSuccess) err = cudaStreamSynchronize(stream);
  if (err != cudaSuccess) return done(cuda_fail(err, "copy of y"));
  return done(B200SP_OK);
}

int spmv_csr_host(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, const void* vals, const void* x,
                  void* y, float alpha, float beta, int dtype, void* stream) {
  return host_call(false, m, n, nnz, 1, row_ptr, col_idx, vals, x, y, alpha, beta, dtype, stream);
}
int spmm_csr_host(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* row_ptr, const int32_t* col_idx, const void* vals,
                  const void* B, void* Y, float alpha, float beta, int dtype, void* stream) {
  return host_call(true, m, n, nnz, k, row_ptr, col_idx, vals, B, Y, alpha, beta, dtype, stream);
}

int b200sp_validate_csr(int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, const int32_t* col_idx, void* stream_v) {
  int rc = check_sizes(m, n, nnz);
  if (rc != B200SP_OK) return rc;
  if (!row_ptr || (nnz > 0 && !col_idx)) return B200SP_ERR_INVALID_ARG;
  DeviceInfo* dev = nullptr;
  rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  cudaStream_t stream = (cudaStream_t)stream_v;
  int* d_bad = nullptr;
  int h_bad = 0;
  rc = pool_alloc(dev, (void**)&d_bad, 256, stream);
  if (rc != B200SP_OK) return rc;
  cudaError_t e = cudaMemsetAsync(d_bad, 0, sizeof(int), stream);
  if (e == cudaSuccess) {
    validate_csr_kernel<<<dev->sms * 8, 256, 0, stream>>>(row_ptr, col_idx, (int)m, (int)n, (int)nnz, d_bad);
    g_launches++;
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&h_bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, stream);
  cudaFreeAsync(d_bad, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail(e, "b200sp_validate_csr");
  return h_bad ? B200SP_ERR_BAD_CSR : B200SP_OK;
}

// Drops what the one-shot entry points cached under this pointer on the current device: plans keyed on a row_ptr
// (device or host address), COO row offsets keyed on a row_idx, CSC transpose plans keyed on a col_ptr.
int b200sp_cache_drop(const void* key_ptr) {
  if (!key_ptr) return B200SP_ERR_INVALID_ARG;
  int dev = 0;
  CU(cudaGetDevice(&dev));
  std::vector<b200sp_plan*> plans;
  std::vector<void*> blocks;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    for (auto it = g_cache.begin(); it != g_cache.end();) {
      if (std::get<0>(it->first) == dev && std::get<1>(it->first) == key_ptr) { plans.push_back(it->second.plan); it = g_cache.erase(it); }
      else ++it;
    }
    for (auto it = g_coo_cache.begin(); it != g_coo_cache.end();) {
      if (std::get<0>(it->first) == dev && std::get<1>(it->first) == key_ptr) { blocks.push_back(it->second.row_ptr); it = g_coo_cache.erase(it); }
      else ++it;
    }
    for (auto it = g_csc_cache.begin(); it != g_csc_cache.end();) {
      if (std::get<0>(it->first) == dev && std::get<1>(it->first) == key_ptr) {
        blocks.push_back(it->second.block);
        it = g_csc_cache.erase(it);
      } else ++it;
    }
  }
  int rc = B200SP_OK;
  for (b200sp_plan* p : plans) { const int r = plan_free(p); if (r != B200SP_OK) rc = r; }
  if (!blocks.empty()) {
    CU(cudaDeviceSynchronize());
    for (void* q : blocks) if (q) cudaFree(q);
  }
  return rc;
}

void b200sp_cache_clear(void) {
  std::lock_guard<std::mutex> lock(g_mutex);
  for (auto& kv : g_cache) plan_free(kv.second.plan);
  g_cache.clear();
  for (auto& kv : g_coo_cache) cudaFree(kv.second.row_ptr);
  g_coo_cache.clear();
  for (auto& kv : g_csc_cache) csc_free(kv.second);
  g_csc_cache.clear();
  int cur = 0;
  const bool have_cur = cudaGetDevice(&cur) == cudaSuccess;
  for (int i = 0; i < 64; ++i) {
    DeviceInfo& d = g_dev[i];
    if (d.pool) cudaMemPoolTrimTo(d.pool, 0);
    if (d.persist_set > 0 && have_cur) {   // give the L2 set aside for the access-policy windows back
      if (cudaSetDevice(i) == cudaSuccess) {
        cudaCtxResetPersistingL2Cache();
        cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, 0);
        d.persist_set = 0;
      }
      cudaSetDevice(cur);
    }
  }
  (void)cudaGetLastError();
}

const char* b200sp_status_string(int s) {
  switch (s) {
    case B200SP_OK: return "ok";
    case B200SP_ERR_INVALID_ARG: return "invalid argument";
    case B200SP_ERR_UNSUPPORTED: return "unsupported";
    case B200SP_ERR_CUDA: return "CUDA call failed";
    case B200SP_ERR_ALLOC: return "allocation failed";
    case B200SP_ERR_ARCH: return "device is not compute capability 10.x (B200)";
    case B200SP_ERR_BAD_CSR: return "CSR arrays are inconsistent";
    case B200SP_ERR_TIMEOUT: return "a kernel gave up on a bounded wait";
    case B200SP_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

int b200sp_check(void* stream_v) {
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  cudaStream_t stream = (cudaStream_t)stream_v;
  int h = 0;
  if (!dev->err_flag) { CU(cudaStreamSynchronize(stream)); return B200SP_OK; }   // no kernel with a bounded wait has run yet
  CU(cudaMemcpyAsync(&h, dev->err_flag, sizeof(int), cudaMemcpyDeviceToHost, stream));
  CU(cudaStreamSynchronize(stream));
  if (h) { CU(cudaMemsetAsync(dev->err_flag, 0, sizeof(int), stream)); CU(cudaStreamSynchronize(stream)); return B200SP_ERR_TIMEOUT; }
  return B200SP_OK;
}

const char* b200sp_last_cuda_error(void) { return g_last_error.c_str(); }
int b200sp_version(void) { return kVersion; }
int b200sp_checked_build(void) {
#ifdef B200SP_BOUNDS_CHECK
  return 1;
#else
  return 0;
#endif
}
int64_t b200sp_launch_count(void) { return g_launches.load(); }

// One row per switch: where it lives and which values it accepts (exactly those listed in b200sp_tuning.h; the test suite
// runs every one of them).  Called with g_mutex held.
static int option_access(const char* name, int* get, const int* set) {
  struct Entry { const char* name; int* slot; bool boolean; std::initializer_list<int> values; int lo, hi; };
  const Entry table[] = {
      {"spmv_kernel", &g_opt.spmv_kernel, false, {-1, 0, 1, 2, 3}, 0, 0},
      {"spmm_bstage", &g_opt.spmm_bstage, true, {}, 0, 0},
      {"spmm_sliced", &g_opt.spmm_sliced, true, {}, 0, 0},
      {"spmm_stage_a", &g_opt.spmm_stage_a, false, {0, 1, 2}, 0, 0},
      {"spmm_flat", &g_opt.spmm_flat, false, {0, 1, 2}, 0, 0},
      {"spmm_ranges", &g_opt.spmm_ranges, false, {0, 1, 2, 3, 4, 8}, 0, 0},
      {"merge_items", &g_opt.merge_items, false, {1024, 2048, 4096}, 0, 0},
      {"merge_threads", &g_opt.merge_threads, false, {64, 128, 256}, 0, 0},
      {"merge_carve", &g_opt.merge_carve, false, {-1, 0, 25, 45, 60, 75, 100}, 0, 0},
      {"merge_short", &g_opt.merge_short, false, {8, 16, 32, 64}, 0, 0},
      {"merge_empty", &g_opt.merge_empty, true, {}, 0, 0},
      {"row_stages", &g_opt.row_stages, false, {2, 3, 4}, 0, 0},
      {"row_ctas", &g_opt.row_ctas, false, {1, 2, 3, 4}, 0, 0},
      {"row_smem_kb", &g_opt.row_smem_kb, false, {48, 96, 160, 220, 227}, 0, 0},
      {"row_threads", &g_opt.row_threads, false, {128, 256}, 0, 0},
      {"row_unroll", &g_opt.row_unroll, false, {8, 16}, 0, 0},
      {"uni_unroll", &g_opt.uni_unroll, false, {0, 1, 2, 4}, 0, 0},
      {"uni_ctas", &g_opt.uni_ctas, false, {0, 1, 2, 4, 8}, 0, 0},
      {"sub_lanes", &g_opt.sub_lanes, false, {0, 1, 2, 4, 8, 16, 32}, 0, 0},
      {"bstage_threads", &g_opt.bstage_threads, false, {256, 512, 1024}, 0, 0},
      {"bstage_nnz", &g_opt.bstage_nnz, false, {0, 16384, 65536, 131072, 524288}, 0, 0},
      {"bstage_stage_a", &g_opt.bstage_stage_a, true, {}, 0, 0},
      {"bstage_quads", &g_opt.bstage_quads, true, {}, 0, 0},
      {"x_l2_window", &g_opt.x_l2_window, true, {}, 0, 0},
      {"pdl", &g_opt.pdl, true, {}, 0, 0},
      {"debug_no_copies", &g_opt.debug_no_copies, true, {}, 0, 0},
      {"log", &g_opt.log, true, {}, 0, 0},
      {"pool_keep_mb", &g_opt.pool_keep_mb, false, {}, 0, 1 << 20},
      {"spin_limit", &g_opt.spin_limit, false, {}, 1, 1 << 30},
      {"fail_alloc_after", &g_opt.fail_alloc_after, false, {}, 0, 1 << 30},
  };
  for (const Entry& e : table) {
    if (strcmp(name, e.name)) continue;
    if (get) { *get = *e.slot; return B200SP_OK; }
    const int value = *set;
    if (e.boolean) { *e.slot = value ? 1 : 0; return B200SP_OK; }
    if (e.values.size()) {
      for (int v : e.values) if (v == value) { *e.slot = value; return B200SP_OK; }
      return B200SP_ERR_INVALID_ARG;
    }
    if (value < e.lo || value > e.hi) return B200SP_ERR_INVALID_ARG;
    *e.slot = value;
    return B200SP_OK;
  }
  return B200SP_ERR_INVALID_ARG;
}

int b200sp_set_option(const char* name, int value) {
  if (!name) return B200SP_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  return option_access(name, nullptr, &value);
}

int b200sp_get_option(const char* name, int* value) {
  if (!name || !value) return B200SP_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  return option_access(name, value, nullptr);
}

}  // extern "C"

// Environment at load time: B200SP_OPTIONS="name=value,name=value" sets switches as b200sp_set_option would (entries that
// are not accepted are reported on stderr and skipped); B200SP_LOG=1 is short for the switch "log" = 1.
namespace {
struct EnvironmentAtLoad {
  EnvironmentAtLoad() {
    if (const char* lg = getenv("B200SP_LOG")) b200sp_set_option("log", atoi(lg));
    const char* opts = getenv("B200SP_OPTIONS");
    if (!opts) return;
    std::string all(opts);
    size_t pos = 0;
    while (pos < all.size()) {
      size_t end = all.find(',', pos);
      if (end == std::string::npos) end = all.size();
      const std::string item = all.substr(pos, end - pos);
      const size_t eq = item.find('=');
      if (eq == std::string::npos || b200sp_set_option(item.substr(0, eq).c_str(), atoi(item.c_str() + eq + 1)) != B200SP_OK)
        fprintf(stderr, "b200sp: B200SP_OPTIONS entry '%s' not accepted\n", item.c_str());
      pos = end + 1;
    }
  }
} g_environment_at_load;
}  // namespace
