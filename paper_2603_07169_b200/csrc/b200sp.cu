// C ABI of libb200sp.so: argument checks, plan pass, kernel selection and launches.
// The operations are those of the paper's Appendix C, Table 6, tasks 12 (SpMV CSR) and 13 (SpMM CSR),
// generalised with alpha / beta; see include/b200sp.h for the contract of every entry point.
#include "../../include/b200sp.h"

#include <atomic>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <tuple>

#include "common.cuh"
#include "plan_kernels.cuh"
#include "spmv_kernels.cuh"
#include "spmm_kernels.cuh"

using namespace b200sp;

namespace {

constexpr int kVersion = 100;  // 0.1.0

// SpMV merge-tile configuration
constexpr int kItems = 4096;
constexpr int kThreads = 256;
constexpr int kShortMax = 32;
// SpMM
constexpr int kSpmmThreads = 256;
constexpr int kSpmmTileNnz = 4096;

thread_local std::string g_last_error;
std::atomic<int64_t> g_launches{0};
std::mutex g_mutex;

struct Options {
  int spmv_kernel = -1;
  int x_l2_window = 1;
} g_opt;

struct DeviceInfo {
  bool known = false;
  int cc_major = 0, sms = 0, persist_max = 0, window_max = 0, l2_bytes = 0;
  size_t persist_set = 0;
};
DeviceInfo g_dev[64];

int cuda_fail(cudaError_t e, const char* what) {
  char buf[512];
  snprintf(buf, sizeof buf, "%s: %s", what, cudaGetErrorString(e));
  g_last_error = buf;
  (void)cudaGetLastError();
  return B200SP_ERR_CUDA;
}
#define CU(call)                                                   \
  do {                                                             \
    cudaError_t e_ = (call);                                       \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call);            \
  } while (0)

int device_info(DeviceInfo** out) {
  int dev = 0;
  CU(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return B200SP_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceInfo& d = g_dev[dev];
  if (!d.known) {
    CU(cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    CU(cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev));
    CU(cudaDeviceGetAttribute(&d.persist_max, cudaDevAttrMaxPersistingL2CacheSize, dev));
    CU(cudaDeviceGetAttribute(&d.window_max, cudaDevAttrMaxAccessPolicyWindowSize, dev));
    CU(cudaDeviceGetAttribute(&d.l2_bytes, cudaDevAttrL2CacheSize, dev));
    d.known = true;
  }
  *out = &d;
  return d.cc_major == 10 ? B200SP_OK : B200SP_ERR_ARCH;
}

// Launch with an optional L2 access-policy window (persisting hits) over the gathered operand.
template <typename... KArgs, typename... Args>
int launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, const void* win_ptr, size_t win_bytes,
           DeviceInfo* dev, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  cfg.attrs = attr;
  cfg.numAttrs = 0;
  if (win_ptr && win_bytes && g_opt.x_l2_window && dev->persist_max > 0 && dev->window_max > 0) {
    size_t want = win_bytes < (size_t)dev->persist_max ? win_bytes : (size_t)dev->persist_max;
    {
      std::lock_guard<std::mutex> lock(g_mutex);
      if (want > dev->persist_set) {
        if (cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want) == cudaSuccess) dev->persist_set = want;
        else (void)cudaGetLastError();
      }
    }
    if (dev->persist_set > 0) {
      const size_t wb = win_bytes < (size_t)dev->window_max ? win_bytes : (size_t)dev->window_max;
      attr[0].id = cudaLaunchAttributeAccessPolicyWindow;
      attr[0].val.accessPolicyWindow.base_ptr = const_cast<void*>(win_ptr);
      attr[0].val.accessPolicyWindow.num_bytes = wb;
      attr[0].val.accessPolicyWindow.hitRatio = wb <= dev->persist_set ? 1.0f : (float)((double)dev->persist_set / (double)wb);
      attr[0].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
      attr[0].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
      cfg.numAttrs = 1;
    }
  }
  CU(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return B200SP_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

int check_sizes(int64_t m, int64_t n, int64_t nnz) {
  const int64_t lim = (int64_t)1 << 31;
  if (m < 0 || n < 0 || nnz < 0 || m >= lim - 1 || n >= lim || nnz >= lim) return B200SP_ERR_INVALID_ARG;
  if (nnz > 0 && (m == 0 || n == 0)) return B200SP_ERR_INVALID_ARG;
  return B200SP_OK;
}

}  // namespace

struct b200sp_plan {
  int device = 0;
  const int32_t* row_ptr = nullptr;
  b200sp_plan_info_t info = {};
  int32_t* split_row = nullptr;       // spmv tiles + 1
  float* carry = nullptr;             // spmv tiles
  float* tail = nullptr;              // spmv tiles
  int32_t* spmm_split_row = nullptr;  // spmm tiles + 1
};

namespace {

std::map<std::tuple<int, const void*, int64_t, int64_t, int64_t>, b200sp_plan*> g_cache;

int plan_free(b200sp_plan* p) {
  if (!p) return B200SP_OK;
  int rc = B200SP_OK;
  for (void* q : {(void*)p->split_row, (void*)p->carry, (void*)p->tail, (void*)p->spmm_split_row})
    if (q) { cudaError_t e = cudaFree(q); if (e != cudaSuccess) rc = cuda_fail(e, "cudaFree"); }
  delete p;
  return rc;
}

int plan_build(b200sp_plan** out, int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, cudaStream_t stream) {
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  b200sp_plan* p = new b200sp_plan();
  CU(cudaGetDevice(&p->device));
  p->row_ptr = row_ptr;
  b200sp_plan_info_t& I = p->info;
  I.m = m; I.n = n; I.nnz = nnz;
  I.spmv_tile_items = kItems;
  I.spmv_tiles = (int32_t)((m + nnz + kItems - 1) / kItems);
  I.spmm_tile_nnz = kSpmmTileNnz;
  I.spmm_tiles = (int32_t)((nnz + kSpmmTileNnz - 1) / kSpmmTileNnz);
  I.spmv_kernel = g_opt.spmv_kernel >= 0 ? g_opt.spmv_kernel : 0;
  if (m == 0) { *out = p; return B200SP_OK; }

  PlanStats* d_stats = nullptr;
  PlanStats h = {};
  h.min_len = 0x7FFFFFFF;
  auto fail = [&](int code) { if (d_stats) cudaFree(d_stats); plan_free(p); return code; };
#define CUP(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(cuda_fail(e_, #call)); } while (0)
  CUP(cudaMalloc(&d_stats, sizeof(PlanStats)));
  CUP(cudaMemcpyAsync(d_stats, &h, sizeof h, cudaMemcpyHostToDevice, stream));
  {
    const int blocks = (int)((m + 256 * 8 - 1) / (256 * 8));
    const int grid = blocks < dev->sms * 8 ? (blocks > 0 ? blocks : 1) : dev->sms * 8;
    plan_stats_kernel<<<grid, 256, 0, stream>>>(row_ptr, (int)m, d_stats);
    g_launches++;
  }
  const size_t nt = (size_t)I.spmv_tiles, ns = (size_t)I.spmm_tiles;
  CUP(cudaMalloc(&p->split_row, (nt + 1) * sizeof(int32_t)));
  CUP(cudaMalloc(&p->carry, (nt + 1) * sizeof(float)));
  CUP(cudaMalloc(&p->tail, (nt + 1) * sizeof(float)));
  CUP(cudaMalloc(&p->spmm_split_row, (ns + 1) * sizeof(int32_t)));
  I.scratch_bytes = (int64_t)((nt + 1) * 12 + (ns + 1) * 4);
  plan_merge_split_kernel<<<(unsigned)((nt + 1 + 255) / 256), 256, 0, stream>>>(row_ptr, (int)m, (int)nnz, kItems, (int)nt, p->split_row);
  plan_nnz_split_kernel<<<(unsigned)((ns + 1 + 255) / 256), 256, 0, stream>>>(row_ptr, (int)m, (int)nnz, kSpmmTileNnz, (int)ns, p->spmm_split_row);
  g_launches += 2;
  CUP(cudaGetLastError());
  CUP(cudaMemcpyAsync(&h, d_stats, sizeof h, cudaMemcpyDeviceToHost, stream));
  CUP(cudaStreamSynchronize(stream));
  CUP(cudaFree(d_stats));
  d_stats = nullptr;
#undef CUP
  if (h.bad) { plan_free(p); return B200SP_ERR_BAD_CSR; }
  I.min_row_len = h.min_len; I.max_row_len = h.max_len;
  for (int j = 0; j < B200SP_NUM_BINS; ++j) { I.bin_rows[j] = (int64_t)h.bin_rows[j]; I.bin_nnz[j] = (int64_t)h.bin_nnz[j]; }
  *out = p;
  return B200SP_OK;
}

template <typename T>
int run_scale(long long count, T* y, float beta, cudaStream_t stream, DeviceInfo* dev) {
  if (count == 0) return B200SP_OK;
  long long blocks = (count + 255) / 256;
  const long long cap = (long long)dev->sms * 16;
  if (blocks > cap) blocks = cap;
  return launch(scale_kernel<T>, dim3((unsigned)blocks), dim3(256), stream, nullptr, 0, dev, count, y, beta);
}

template <typename T>
int run_spmv(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
             cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  if (I.m == 0) return B200SP_OK;
  if (alpha == 0.0f || I.nnz == 0) return run_scale<T>(I.m, y, beta, stream, dev);
  const int tiles = I.spmv_tiles;
  int rc = launch(spmv_merge_tile_kernel<T, kItems, kThreads, kShortMax>, dim3(tiles), dim3(kThreads), stream, x,
                  (size_t)I.n * sizeof(T), dev, (int)I.m, (int)I.nnz, p->row_ptr, col_idx, vals, x, y, alpha, beta,
                  (const int*)p->split_row, p->carry, p->tail);
  if (rc != B200SP_OK) return rc;
  if (tiles > 1)
    rc = launch(spmv_carry_fixup_kernel<T, kItems>, dim3((tiles + 127) / 128), dim3(128), stream, nullptr, 0, dev, tiles,
                p->row_ptr, (const int*)p->split_row, (const float*)p->carry, (const float*)p->tail, y, alpha, beta);
  return rc;
}

template <typename T, int VEC, int LANES, int NCH>
int launch_spmm(const b200sp_plan_info_t& I, const int32_t* row_ptr, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y,
                float alpha, float beta, cudaStream_t stream, DeviceInfo* dev) {
  constexpr int GROUPS = kSpmmThreads / LANES;
  const unsigned grid = (unsigned)((I.m + GROUPS - 1) / GROUPS);
  return launch(spmm_row_group_kernel<T, VEC, LANES, NCH, kSpmmThreads>, dim3(grid), dim3(kSpmmThreads), stream, B,
                (size_t)I.n * k * sizeof(T), dev, (int)I.m, k, row_ptr, col_idx, vals, B, Y, alpha, beta);
}

template <typename T, int VEC>
int run_spmm(b200sp_plan* p, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y, float alpha, float beta,
             cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  if (I.m == 0) return B200SP_OK;
  if (alpha == 0.0f || I.nnz == 0) return run_scale<T>((long long)I.m * k, Y, beta, stream, dev);
  if (k % VEC != 0) {  // ragged k: scalar lanes
    if (k <= 8) return launch_spmm<T, 1, 8, 1>(I, p->row_ptr, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
    return launch_spmm<T, 1, 32, 2>(I, p->row_ptr, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  }
  const int vecs = k / VEC;  // vector columns per row
  if (vecs <= 4) return launch_spmm<T, VEC, 4, 1>(I, p->row_ptr, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  if (vecs <= 8) return launch_spmm<T, VEC, 8, 1>(I, p->row_ptr, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  if (vecs <= 16) return launch_spmm<T, VEC, 16, 1>(I, p->row_ptr, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  if (vecs <= 32) return launch_spmm<T, VEC, 32, 1>(I, p->row_ptr, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
  return launch_spmm<T, VEC, 32, 2>(I, p->row_ptr, k, col_idx, vals, B, Y, alpha, beta, stream, dev);
}

int check_common(const b200sp_plan* p, const void* col_idx, const void* vals, const void* dense_in, const void* dense_out, int dtype) {
  if (!p) return B200SP_ERR_INVALID_ARG;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  const b200sp_plan_info_t& I = p->info;
  if (I.nnz > 0 && (!col_idx || !vals || !dense_in)) return B200SP_ERR_INVALID_ARG;
  if (I.m > 0 && !dense_out) return B200SP_ERR_INVALID_ARG;
  if (!aligned16(col_idx) || !aligned16(vals) || !aligned16(dense_in) || !aligned16(dense_out)) return B200SP_ERR_INVALID_ARG;
  return B200SP_OK;
}

int get_cached_plan(b200sp_plan** out, int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, cudaStream_t stream) {
  int dev = 0;
  CU(cudaGetDevice(&dev));
  const auto key = std::make_tuple(dev, (const void*)row_ptr, m, n, nnz);
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    auto it = g_cache.find(key);
    if (it != g_cache.end()) { *out = it->second; return B200SP_OK; }
  }
  b200sp_plan* p = nullptr;
  int rc = b200sp_plan_create(&p, m, n, nnz, row_ptr, stream);
  if (rc != B200SP_OK) return rc;
  std::lock_guard<std::mutex> lock(g_mutex);
  auto ins = g_cache.emplace(key, p);
  if (!ins.second) { plan_free(p); p = ins.first->second; }
  *out = p;
  return B200SP_OK;
}

}  // namespace

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
  CU(cudaMallocAsync((void**)&base, total, stream));
  char* d_rp = base; char* d_ci = d_rp + up(b_rp); char* d_va = d_ci + up(b_ci); char* d_in = d_va + up(b_va); char* d_out = d_in + up(b_in);
  b200sp_plan* p = nullptr;
  auto done = [&](int code) { if (p) plan_free(p); cudaFreeAsync(base, stream); cudaStreamSynchronize(stream); return code; };
#define CUH(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return done(cuda_fail(e_, #call)); } while (0)
  CUH(cudaMemcpyAsync(d_rp, row_ptr, b_rp, cudaMemcpyHostToDevice, stream));
  if (nnz > 0) {
    CUH(cudaMemcpyAsync(d_ci, col_idx, b_ci, cudaMemcpyHostToDevice, stream));
    CUH(cudaMemcpyAsync(d_va, vals, b_va, cudaMemcpyHostToDevice, stream));
    CUH(cudaMemcpyAsync(d_in, in, b_in, cudaMemcpyHostToDevice, stream));
  }
  if (beta != 0.0f) CUH(cudaMemcpyAsync(d_out, out, b_out, cudaMemcpyHostToDevice, stream));
  rc = plan_build(&p, m, n, nnz, (const int32_t*)d_rp, stream);
  if (rc != B200SP_OK) { p = nullptr; return done(rc); }
  rc = is_mm ? b200sp_spmm(p, k, (const int32_t*)d_ci, d_va, d_in, d_out, alpha, beta, dtype, stream)
             : b200sp_spmv(p, (const int32_t*)d_ci, d_va, d_in, d_out, alpha, beta, dtype, stream);
  if (rc != B200SP_OK) return done(rc);
  CUH(cudaMemcpyAsync(out, d_out, b_out, cudaMemcpyDeviceToHost, stream));
  CUH(cudaStreamSynchronize(stream));
#undef CUH
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
  CU(cudaMalloc(&d_bad, sizeof(int)));
  cudaError_t e = cudaMemsetAsync(d_bad, 0, sizeof(int), stream);
  if (e == cudaSuccess) {
    validate_csr_kernel<<<dev->sms * 8, 256, 0, stream>>>(row_ptr, col_idx, (int)m, (int)n, (int)nnz, d_bad);
    g_launches++;
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&h_bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  cudaFree(d_bad);
  if (e != cudaSuccess) return cuda_fail(e, "b200sp_validate_csr");
  return h_bad ? B200SP_ERR_BAD_CSR : B200SP_OK;
}

void b200sp_cache_clear(void) {
  std::lock_guard<std::mutex> lock(g_mutex);
  for (auto& kv : g_cache) plan_free(kv.second);
  g_cache.clear();
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
    default: return "unknown status";
  }
}

const char* b200sp_last_cuda_error(void) { return g_last_error.c_str(); }
int b200sp_version(void) { return kVersion; }
int64_t b200sp_launch_count(void) { return g_launches.load(); }

int b200sp_set_option(const char* name, int value) {
  if (!name) return B200SP_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!strcmp(name, "spmv_kernel")) { if (value < -1 || value > 1) return B200SP_ERR_INVALID_ARG; g_opt.spmv_kernel = value; return B200SP_OK; }
  if (!strcmp(name, "x_l2_window")) { g_opt.x_l2_window = value ? 1 : 0; return B200SP_OK; }
  return B200SP_ERR_INVALID_ARG;
}

}  // extern "C"
