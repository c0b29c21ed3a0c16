// C ABI of libb200sp.so: argument checks, plan pass, kernel selection and launches.
// The operations are those of the paper's Appendix C, Table 6, tasks 12 (SpMV CSR) and 13 (SpMM CSR),
// generalised with alpha / beta; see include/b200sp.h for the contract of every entry point.
#include "../../include/b200sp.h"

#include <atomic>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <algorithm>
#include <string>
#include <vector>
#include <tuple>

#include "common.cuh"
#include "plan_kernels.cuh"
#include "spmv_kernels.cuh"
#include "spmv_row_kernels.cuh"
#include "spmv_uniform_kernels.cuh"
#include "spmv_merge_stage_kernels.cuh"
#include "spmm_kernels.cuh"
#include "spmm_bstage_kernels.cuh"
#include "format_kernels.cuh"

using namespace b200sp;

namespace {

constexpr int kVersion = 100;  // 0.1.0

// SpMV merge-tile configuration
constexpr int kItems = 4096;
constexpr int kThreads = 256;
constexpr int kShortMax = 32;
// SpMV row-direct kernel: eligibility and shared-memory budget (two CTAs per SM)
constexpr int kRowThreads = 256;
constexpr int kRowMaxLen = 64;
constexpr int kSmemPerSm = 227 * 1024;   // usable shared memory per SM (each CTA also reserves 1 KB)
// SpMM
constexpr int kSpmmThreads = 256;
constexpr int kSpmmTileNnz = 4096;
constexpr int kSmallNnz = 1 << 20;   // at or below this many nonzeros SpMV uses the sub-warp-per-row kernel
constexpr int kLongRow = 1024;   // rows longer than this get a CTA of their own in SpMM (last length bin of the plan)

thread_local std::string g_last_error;
std::atomic<int64_t> g_launches{0};
std::mutex g_mutex;

struct Options {
  int spmv_kernel = -1;
  int x_l2_window = 0;   // measured: no gain on the large workloads (x stays in L2 anyway), +1.4 us per launch on tiny ones
  int row_stages = 2;   // shared-memory stages per CTA of the row-direct kernel (2..4)
  int row_ctas = 3;     // CTAs per SM the row-direct kernel is sized for (1..4)
  int row_unroll = 8;   // gathers in flight per thread (8 or 16)
  int row_smem_kb = 220;  // shared memory per SM the row-direct kernel may use for its stages (the rest stays L1)
  int row_threads = 256;  // threads per CTA of the row-direct kernel (128 or 256)
  int uni_unroll = 2;     // groups of four nonzeros in flight per thread of the uniform-row kernel (1, 2 or 4)
  int uni_ctas = 0;       // CTAs per SM for the uniform-row kernel (0 = as many as fit)
  int merge_staged = 0;   // 1 = persistent staged merge kernel, 0 = one-tile-per-CTA merge kernel
  int merge_items = 2048; // merge items per tile (2048 or 4096)
  int merge_stages = 3;   // shared-memory stages per CTA of the staged merge kernel (2..4)
  int merge_ctas = 2;     // CTAs per SM of the staged merge kernel
  int merge_threads = 128; // threads per CTA of the one-tile-per-CTA merge kernel (128 or 256)
  int bstage_threads = 1024; // threads per CTA of that kernel (256, 512 or 1024)
  int bstage_nnz = 131072;   // nonzeros per CTA it aims for
  int spmm_bstage = 1;     // 1 = hold the slice of B in shared memory when A has few columns (default), 0 = never
  int spmm_sliced = 1;     // 1 = k-sliced SpMM kernel (default), 0 = one pass over all of k
  int sub_lanes = 0;       // lanes per row of the sub-warp kernel (0 = from the mean row length)
  int merge_short = 32;    // rows up to this many products are added by one thread (8, 16, 32, 64)
  int merge_carve = 30;    // shared-memory carveout (percent) requested for it, -1 = leave to the driver
} g_opt;

struct DeviceInfo {
  bool known = false;
  int cc_major = 0, sms = 0, persist_max = 0, window_max = 0, l2_bytes = 0;
  size_t persist_set = 0;
  int* err_flag = nullptr;  // device int: set by a kernel whose bounded wait ran out
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

// The flag that kernels with bounded waits raise; allocated on first use (those kernels only).
int ensure_err_flag(DeviceInfo* d) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!d->err_flag) {
    CU(cudaMalloc(&d->err_flag, sizeof(int)));
    CU(cudaMemset(d->err_flag, 0, sizeof(int)));
  }
  return B200SP_OK;
}

// Launch with an optional L2 access-policy window (persisting hits) over the gathered operand.
template <typename... KArgs, typename... Args>
int launch_smem(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, const void* win_ptr,
                size_t win_bytes, DeviceInfo* dev, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
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

template <typename... KArgs, typename... Args>
int launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, const void* win_ptr, size_t win_bytes,
           DeviceInfo* dev, Args... args) {
  return launch_smem(kernel, grid, block, 0, stream, win_ptr, win_bytes, dev, args...);
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
  int32_t* long_rows = nullptr;       // rows longer than kLongRow, ascending
  int num_long = 0;
  const void* probed_col_idx = nullptr;   // col_idx the column-locality probe last ran on
  bool cols_local = true;                 // its verdict: adjacent rows share most of their lines of x
};

namespace {

std::map<std::tuple<int, const void*, int64_t, int64_t, int64_t>, b200sp_plan*> g_cache;

int plan_free(b200sp_plan* p) {
  if (!p) return B200SP_OK;
  int rc = B200SP_OK;
  for (void* q : {(void*)p->split_row, (void*)p->carry, (void*)p->tail, (void*)p->spmm_split_row, (void*)p->long_rows})
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
  const int items = g_opt.merge_items == 4096 ? 4096 : (g_opt.merge_items == 1024 ? 1024 : 2048);
  I.spmv_tile_items = items;
  I.spmv_tiles = (int32_t)((m + nnz + items - 1) / items);
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
  plan_merge_split_kernel<<<(unsigned)((nt + 1 + 255) / 256), 256, 0, stream>>>(row_ptr, (int)m, (int)nnz, items, (int)nt, p->split_row);
  plan_nnz_split_kernel<<<(unsigned)((ns + 1 + 255) / 256), 256, 0, stream>>>(row_ptr, (int)m, (int)nnz, kSpmmTileNnz, (int)ns, p->spmm_split_row);
  g_launches += 2;
  CUP(cudaGetLastError());
  CUP(cudaMemcpyAsync(&h, d_stats, sizeof h, cudaMemcpyDeviceToHost, stream));
  CUP(cudaStreamSynchronize(stream));
  CUP(cudaFree(d_stats));
  d_stats = nullptr;
  if (!h.bad && h.bin_rows[4] > 0) {   // list of the rows in the last length bin (> kLongRow), sorted on the host
    const int cap = (int)h.bin_rows[4];
    int* d_count = nullptr;
    CUP(cudaMalloc(&p->long_rows, (size_t)cap * sizeof(int32_t)));
    CUP(cudaMalloc(&d_count, sizeof(int)));
    cudaError_t e = cudaMemsetAsync(d_count, 0, sizeof(int), stream);
    if (e == cudaSuccess) {
      const int blocks = (int)((m + 255) / 256);
      plan_long_rows_kernel<<<blocks < dev->sms * 8 ? blocks : dev->sms * 8, 256, 0, stream>>>(row_ptr, (int)m, kLongRow, cap, p->long_rows, d_count);
      g_launches++;
      e = cudaGetLastError();
    }
    std::vector<int32_t> tmp((size_t)cap);
    if (e == cudaSuccess) e = cudaMemcpyAsync(tmp.data(), p->long_rows, (size_t)cap * sizeof(int32_t), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e == cudaSuccess) { std::sort(tmp.begin(), tmp.end()); e = cudaMemcpyAsync(p->long_rows, tmp.data(), (size_t)cap * sizeof(int32_t), cudaMemcpyHostToDevice, stream); }
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    cudaFree(d_count);
    if (e != cudaSuccess) return fail(cuda_fail(e, "plan long-row list"));
    p->num_long = cap;
    I.scratch_bytes += (int64_t)cap * 4;
  }
#undef CUP
  if (h.bad) { plan_free(p); return B200SP_ERR_BAD_CSR; }
  I.min_row_len = h.min_len; I.max_row_len = h.max_len;
  for (int j = 0; j < B200SP_NUM_BINS; ++j) { I.bin_rows[j] = (int64_t)h.bin_rows[j]; I.bin_nnz[j] = (int64_t)h.bin_nnz[j]; }
  // Kernel choice from the row statistics: when every row is short and the mean is not far below the
  // maximum, a thread per row wastes little and rows never need splitting -> row-direct kernel.
  // Anything with long or very uneven rows goes to the merge-tile kernel.
  const bool row_direct_ok = nnz > 0 && h.max_len <= kRowMaxLen && aligned16(row_ptr) &&
                             (h.max_len <= 8 || nnz * 4 >= (int64_t)h.max_len * m);
  // Rows all of one length 4, 8, ..., 128: sub-warp-per-row kernel with 128-bit loads and no shared memory.
  const bool uniform_ok = nnz > 0 && h.min_len == h.max_len && h.max_len >= 4 && h.max_len <= 128 && (h.max_len & (h.max_len - 1)) == 0;
  const bool row_direct_possible = nnz > 0 && h.max_len <= kRowMaxLen && aligned16(row_ptr);
  int choice = uniform_ok ? 2 : (row_direct_ok ? 1 : 0);
  // Small problems (launch-latency regime): one sub-warp per row, no scratch, maximum spread over the SMs -- unless the
  // rows are uniform (the uniform-row kernel is as flat) or the row-direct kernel would still get a tile for every SM.
  if (nnz > 0 && nnz <= kSmallNnz && h.max_len <= 4096 && !uniform_ok && !(row_direct_ok && m >= (int64_t)kRowThreads * dev->sms)) choice = 3;
  if (g_opt.spmv_kernel == 3) choice = h.max_len <= 65536 ? 3 : 0;
  if (g_opt.spmv_kernel == 0) choice = 0;
  if (g_opt.spmv_kernel == 1) choice = row_direct_possible ? 1 : 0;
  if (g_opt.spmv_kernel == 2) choice = uniform_ok ? 2 : (row_direct_ok ? 1 : 0);
  I.spmv_kernel = choice;
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

int gcd_int(int a, int b) { while (b) { const int t = a % b; a = b; b = t; } return a; }

template <typename T, int THREADS, int UNROLL, bool ROT>
int launch_row_direct(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                      cudaStream_t stream, DeviceInfo* dev, int rot_lanes) {
  const b200sp_plan_info_t& I = p->info;
  const int max_len = I.max_row_len > 0 ? I.max_row_len : 1;
  const int stages = g_opt.row_stages, ctas = g_opt.row_ctas;
  int sm_budget = g_opt.row_smem_kb * 1024;
  if (sm_budget > kSmemPerSm) sm_budget = kSmemPerSm;
  const int cta_budget = sm_budget / ctas - 1024 - 256;
  const int stage_budget = cta_budget / stages;
  const int cap_max = (stage_budget - (THREADS + 4) * 4 - 64) / (4 + (int)sizeof(T));
  int R = (cap_max - 16) / max_len;
  if (R > THREADS) R = THREADS;
  R &= ~3;
  if (R < 4) return B200SP_ERR_UNSUPPORTED;
  const int cap = (R * max_len + 16 + 7) & ~7;
  const int tiles = (int)((I.m + R - 1) / R);
  const size_t smem = (size_t)stages * row_tile_stage_bytes<T>(R, cap);
  auto kernel = spmv_row_tile_kernel<T, THREADS, UNROLL, ROT>;
  static int configured[64] = {};   // per instantiation and device: the carveout last set (percent + 1)
  int carve = (int)(((size_t)ctas * (smem + 1024 + 128) * 100 + (size_t)kSmemPerSm) / ((size_t)kSmemPerSm + 1024)) + 1;
  if (carve > 100) carve = 100;
  if (configured[p->device] != carve + 1) {
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerSm - 1024));
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, carve));
    configured[p->device] = carve + 1;
  }
  const int grid = tiles < ctas * dev->sms ? tiles : ctas * dev->sms;
  const int rc_flag = ensure_err_flag(dev);
  if (rc_flag != B200SP_OK) return rc_flag;
  return launch_smem(kernel, dim3(grid), dim3(THREADS), smem, stream, x, (size_t)I.n * sizeof(T), dev, (int)I.m, (int)I.nnz,
                     p->row_ptr, col_idx, vals, x, y, alpha, beta, R, cap, tiles, stages, rot_lanes, dev->err_flag, 0);
}

// The same kernel on an ELL matrix of at most kRowMaxLen slots per row (implicit row offsets, padding skipped).
template <typename T>
int launch_row_direct_ell(int64_t m, int width, const int32_t* col_ids, const T* vals, const T* x, T* y, float alpha, float beta,
                          cudaStream_t stream, DeviceInfo* dev) {
  constexpr int THREADS = kRowThreads, UNROLL = 8;
  const int stages = g_opt.row_stages, ctas = g_opt.row_ctas;
  int sm_budget = g_opt.row_smem_kb * 1024;
  if (sm_budget > kSmemPerSm) sm_budget = kSmemPerSm;
  const int stage_budget = (sm_budget / ctas - 1024 - 256) / stages;
  const int cap_max = (stage_budget - (THREADS + 4) * 4 - 64) / (4 + (int)sizeof(T));
  int R = (cap_max - 16) / width;
  if (R > THREADS) R = THREADS;
  R &= ~3;
  if (R < 4) return B200SP_ERR_UNSUPPORTED;
  const int cap = (R * width + 16 + 7) & ~7;
  const int tiles = (int)((m + R - 1) / R);
  const size_t smem = (size_t)stages * row_tile_stage_bytes<T>(R, cap);
  auto kernel = spmv_row_tile_kernel<T, THREADS, UNROLL, false, true>;
  int d = 0;
  CU(cudaGetDevice(&d));
  static int configured[64] = {};
  int carve = (int)(((size_t)ctas * (smem + 1024 + 128) * 100 + (size_t)kSmemPerSm) / ((size_t)kSmemPerSm + 1024)) + 1;
  if (carve > 100) carve = 100;
  if (configured[d] != carve + 1) {
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerSm - 1024));
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, carve));
    configured[d] = carve + 1;
  }
  const int grid = tiles < ctas * dev->sms ? tiles : ctas * dev->sms;
  const int rc_flag = ensure_err_flag(dev);
  if (rc_flag != B200SP_OK) return rc_flag;
  return launch_smem(kernel, dim3(grid), dim3(THREADS), smem, stream, nullptr, 0, dev, (int)m, (int)(m * width), (const int*)nullptr, col_ids,
                     vals, x, y, alpha, beta, R, cap, tiles, stages, 0, dev->err_flag, width);
}

template <typename T>
int run_spmv_row_direct(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                        cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  // equal-length rows: start each lane's walk at a different offset so that a warp's shared-memory reads spread over the banks
  int rot_lanes = 0;
  if (I.min_row_len == I.max_row_len && I.max_row_len > 1) {
    const int g = gcd_int(I.max_row_len, 32);
    if (g > 1) rot_lanes = 32 / g;
  }
#define ROW_DISPATCH(TH, U)                                                                                              \
  return rot_lanes ? launch_row_direct<T, TH, U, true>(p, col_idx, vals, x, y, alpha, beta, stream, dev, rot_lanes)    \
                   : launch_row_direct<T, TH, U, false>(p, col_idx, vals, x, y, alpha, beta, stream, dev, 0)
  if (g_opt.row_threads == 128) {
    if (g_opt.row_unroll == 16) { ROW_DISPATCH(128, 16); }
    ROW_DISPATCH(128, 8);
  }
  if (g_opt.row_unroll == 16) { ROW_DISPATCH(256, 16); }
  ROW_DISPATCH(256, 8);
#undef ROW_DISPATCH
}

template <typename T, int LPR, int UNROLL>
int launch_uniform(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                   cudaStream_t stream, DeviceInfo* dev) {
  constexpr int THREADS = 256;
  const b200sp_plan_info_t& I = p->info;
  auto kernel = spmv_uniform_vec_kernel<T, LPR, UNROLL, THREADS>;
  static int per_sm[64] = {};   // per instantiation and device
  if (!per_sm[p->device]) {
    CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 0));   // all of the unified cache as L1
    int nb = 0;
    CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kernel, THREADS, 0));
    per_sm[p->device] = nb > 0 ? nb : 1;
  }
  const int ctas = g_opt.uni_ctas > 0 && g_opt.uni_ctas < per_sm[p->device] ? g_opt.uni_ctas : per_sm[p->device];
  const long long quads = I.nnz / 4;
  long long blocks = (quads + (long long)THREADS * UNROLL - 1) / ((long long)THREADS * UNROLL);
  const long long cap = (long long)dev->sms * ctas;
  if (blocks > cap) blocks = cap;
  return launch(kernel, dim3((unsigned)blocks), dim3(THREADS), stream, x, (size_t)I.n * sizeof(T), dev, quads, col_idx, vals, x, y, alpha, beta);
}

template <typename T, int LPR>
int run_spmv_uniform_u(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                       cudaStream_t stream, DeviceInfo* dev) {
  if (g_opt.uni_unroll == 1) return launch_uniform<T, LPR, 1>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (g_opt.uni_unroll == 4) return launch_uniform<T, LPR, 4>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  return launch_uniform<T, LPR, 2>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
}

template <typename T>
int run_spmv_uniform(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                     cudaStream_t stream, DeviceInfo* dev) {
  switch (p->info.max_row_len / 4) {
    case 1: return run_spmv_uniform_u<T, 1>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 2: return run_spmv_uniform_u<T, 2>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 4: return run_spmv_uniform_u<T, 4>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 8: return run_spmv_uniform_u<T, 8>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 16: return run_spmv_uniform_u<T, 16>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 32: return run_spmv_uniform_u<T, 32>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  }
  return B200SP_ERR_UNSUPPORTED;
}

template <typename T, int ITEMS, int SHORT = kShortMax>
int run_spmv_merge(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                   cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  const int tiles = I.spmv_tiles;
  int rc;
  if (g_opt.merge_staged) {
    const int stages = g_opt.merge_stages, ctas = g_opt.merge_ctas;
    auto kernel = spmv_merge_stage_kernel<T, ITEMS, kThreads, kShortMax>;
    const size_t smem = (size_t)stages * merge_stage_bytes<T>(ITEMS);
    if ((size_t)ctas * (smem + 2048) > (size_t)kSmemPerSm) return B200SP_ERR_UNSUPPORTED;
    static int configured[64] = {};
    int carve = (int)(((size_t)ctas * (smem + 2048) * 100 + (size_t)kSmemPerSm) / ((size_t)kSmemPerSm + 1024)) + 1;
    if (carve > 100) carve = 100;
    if (configured[p->device] != carve + 1) {
      CU(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerSm - 2048));
      CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, carve));
      configured[p->device] = carve + 1;
    }
    rc = ensure_err_flag(dev);
    if (rc != B200SP_OK) return rc;
    const int grid = tiles < ctas * dev->sms ? tiles : ctas * dev->sms;
    rc = launch_smem(kernel, dim3(grid), dim3(kThreads), smem, stream, x, (size_t)I.n * sizeof(T), dev, (int)I.m, (int)I.nnz, p->row_ptr,
                     col_idx, vals, x, y, alpha, beta, (const int*)p->split_row, p->carry, p->tail, tiles, stages, dev->err_flag);
  } else if (g_opt.merge_threads == 64) {
    auto kernel = spmv_merge_tile_kernel<T, ITEMS, 64, SHORT>;
    if (g_opt.merge_carve >= 0) CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, g_opt.merge_carve));
    rc = launch(kernel, dim3(tiles), dim3(64), stream, x, (size_t)I.n * sizeof(T), dev, (int)I.m, (int)I.nnz, p->row_ptr, col_idx,
                vals, x, y, alpha, beta, (const int*)p->split_row, p->carry, p->tail);
  } else if (g_opt.merge_threads == 128) {
    auto kernel = spmv_merge_tile_kernel<T, ITEMS, 128, SHORT>;
    if (g_opt.merge_carve >= 0) CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, g_opt.merge_carve));
    rc = launch(kernel, dim3(tiles), dim3(128), stream, x, (size_t)I.n * sizeof(T), dev, (int)I.m, (int)I.nnz, p->row_ptr, col_idx,
                vals, x, y, alpha, beta, (const int*)p->split_row, p->carry, p->tail);
  } else {
    auto kernel = spmv_merge_tile_kernel<T, ITEMS, kThreads, kShortMax>;
    if (g_opt.merge_carve >= 0) CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, g_opt.merge_carve));
    rc = launch(kernel, dim3(tiles), dim3(kThreads), stream, x, (size_t)I.n * sizeof(T), dev, (int)I.m, (int)I.nnz, p->row_ptr, col_idx,
                vals, x, y, alpha, beta, (const int*)p->split_row, p->carry, p->tail);
  }
  if (rc != B200SP_OK) return rc;
  if (tiles > 1)
    rc = launch(spmv_carry_fixup_kernel<T, ITEMS>, dim3((tiles + 127) / 128), dim3(128), stream, nullptr, 0, dev, tiles,
                p->row_ptr, (const int*)p->split_row, (const float*)p->carry, (const float*)p->tail, y, alpha, beta);
  return rc;
}

template <typename T, int LPR>
int launch_subwarp(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                   cudaStream_t stream, DeviceInfo* dev) {
  constexpr int THREADS = 128;
  const b200sp_plan_info_t& I = p->info;
  const long long groups_per_cta = THREADS / LPR;
  const long long blocks = (I.m + groups_per_cta - 1) / groups_per_cta;
  if (blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  return launch(spmv_subwarp_kernel<T, LPR, THREADS>, dim3((unsigned)blocks), dim3(THREADS), stream, x, (size_t)I.n * sizeof(T), dev,
                (int)I.m, p->row_ptr, col_idx, vals, x, y, alpha, beta);
}

template <typename T>
int run_spmv_subwarp(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                     cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  const double mean = I.m > 0 ? (double)I.nnz / (double)I.m : 0.0;
  int lpr = g_opt.sub_lanes;
  if (lpr <= 0) lpr = mean <= 3 ? 1 : mean <= 6 ? 2 : mean <= 12 ? 4 : mean <= 24 ? 8 : mean <= 64 ? 16 : 32;
  switch (lpr) {
    case 1: return launch_subwarp<T, 1>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 2: return launch_subwarp<T, 2>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 4: return launch_subwarp<T, 4>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 8: return launch_subwarp<T, 8>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 16: return launch_subwarp<T, 16>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    default: return launch_subwarp<T, 32>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  }
}

// The row-direct kernel gives its shared memory to stages and leaves little L1; that pays only when the gather of x is
// local (adjacent rows share lines).  The first call with a given col_idx samples that property (one small kernel, one
// synchronisation); matrices with scattered columns go to the merge-tile kernel instead.
int probe_col_locality(b200sp_plan* p, const int32_t* col_idx, cudaStream_t stream) {
  if (p->probed_col_idx == (const void*)col_idx) return B200SP_OK;
  const b200sp_plan_info_t& I = p->info;
  unsigned long long* d_out = nullptr;
  unsigned long long h[2] = {0, 0};
  CU(cudaMalloc(&d_out, sizeof h));
  cudaError_t e = cudaMemsetAsync(d_out, 0, sizeof h, stream);
  const int samples = I.m - 1 < 8192 ? (int)(I.m - 1) : 8192;
  if (e == cudaSuccess && samples > 0) {
    plan_col_locality_kernel<<<(samples + 127) / 128, 128, 0, stream>>>(p->row_ptr, col_idx, (int)I.m, samples, d_out);
    g_launches++;
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(h, d_out, sizeof h, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  cudaFree(d_out);
  if (e != cudaSuccess) return cuda_fail(e, "column-locality probe");
  p->cols_local = h[1] == 0 || 2 * h[0] >= h[1];   // at least half of the sampled entries re-use a line of the row above
  p->probed_col_idx = col_idx;
  return B200SP_OK;
}

template <typename T>
int run_spmv(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
             cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  if (I.m == 0) return B200SP_OK;
  if (alpha == 0.0f || I.nnz == 0) return run_scale<T>(I.m, y, beta, stream, dev);
  if (I.spmv_kernel == 1 && g_opt.spmv_kernel != 1) {   // chosen from the row statistics, not forced: confirm with the column probe
    const int rc = probe_col_locality(p, col_idx, stream);
    if (rc != B200SP_OK) return rc;
    if (!p->cols_local) {
      if (I.spmv_tile_items == 4096) return run_spmv_merge<T, 4096>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
      if (I.spmv_tile_items == 1024) return run_spmv_merge<T, 1024>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
      return run_spmv_merge<T, 2048>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    }
  }
  if (I.spmv_kernel == 3) return run_spmv_subwarp<T>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (I.spmv_kernel == 2) return run_spmv_uniform<T>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (I.spmv_kernel == 1) return run_spmv_row_direct<T>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (I.spmv_tile_items == 4096) return run_spmv_merge<T, 4096>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (I.spmv_tile_items == 1024) return run_spmv_merge<T, 1024>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (g_opt.merge_short == 8) return run_spmv_merge<T, 2048, 8>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (g_opt.merge_short == 16) return run_spmv_merge<T, 2048, 16>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (g_opt.merge_short == 64) return run_spmv_merge<T, 2048, 64>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  return run_spmv_merge<T, 2048>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
}

template <typename T, int VEC, int LANES, int NCH>
int launch_spmm(const b200sp_plan_info_t& I, const int32_t* row_ptr, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y,
                float alpha, float beta, cudaStream_t stream, DeviceInfo* dev) {
  constexpr int GROUPS = kSpmmThreads / LANES;
  const unsigned grid = (unsigned)((I.m + GROUPS - 1) / GROUPS);
  return launch(spmm_row_group_kernel<T, VEC, LANES, NCH, kSpmmThreads>, dim3(grid), dim3(kSpmmThreads), stream, B,
                (size_t)I.n * k * sizeof(T), dev, (int)I.m, k, row_ptr, col_idx, vals, B, Y, alpha, beta);
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
  const size_t smem = (size_t)boxes * box_rows * ROW_BYTES;
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
  long long chunks = (I.nnz + g_opt.bstage_nnz - 1) / g_opt.bstage_nnz;   // a given number of nonzeros per CTA ...
  const long long fill = (2LL * dev->sms + slices - 1) / slices;   // ... but at least two CTAs per SM over the grid
  if (chunks < fill) chunks = fill;
  if (chunks > I.m) chunks = I.m;
  if (chunks < 1) chunks = 1;
  const int rows_per_chunk = (int)((I.m + chunks - 1) / chunks);
  const int row_chunks = (int)((I.m + rows_per_chunk - 1) / rows_per_chunk);
  if ((long long)slices * row_chunks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
  int rc = ensure_err_flag(dev);
  if (rc != B200SP_OK) return rc;
  return launch_smem(kernel, dim3((unsigned)(slices * row_chunks)), dim3(THREADS), smem, stream, nullptr, 0, dev, map, (int)I.m, (int)I.n,
                     k, row_chunks, rows_per_chunk, box_rows, p->row_ptr, col_idx, vals, Y, alpha, beta, dev->err_flag);
}

template <typename T, int VEC>
int run_spmm(b200sp_plan* p, int k, const int32_t* col_idx, const T* vals, const T* B, T* Y, float alpha, float beta,
             cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  if (I.m == 0) return B200SP_OK;
  if (alpha == 0.0f || I.nnz == 0) return run_scale<T>((long long)I.m * k, Y, beta, stream, dev);
  if (k % VEC == 0 && g_opt.spmm_bstage && I.nnz >= 4 * I.n && ((size_t)k * sizeof(T)) % 16 == 0) {
    // widest slice of B (128, 64 or 32 bytes per row) whose n rows fit in one SM's shared memory
    const size_t budget = (size_t)kSmemPerSm - 4096;
    const size_t n_pad = (size_t)((I.n + 255) / 256) * 256;
    EncodeTiledFn encode = tensor_map_encoder();
    if (encode && n_pad * 32 <= budget) {
      int rc;
      if (g_opt.bstage_threads == 256) {
        if (n_pad * 128 <= budget) rc = launch_spmm_bstage<T, VEC, 8, 256>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
        else if (n_pad * 64 <= budget) rc = launch_spmm_bstage<T, VEC, 4, 256>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
        else rc = launch_spmm_bstage<T, VEC, 2, 256>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
      } else if (g_opt.bstage_threads == 512) {
        if (n_pad * 128 <= budget) rc = launch_spmm_bstage<T, VEC, 8, 512>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
        else if (n_pad * 64 <= budget) rc = launch_spmm_bstage<T, VEC, 4, 512>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
        else rc = launch_spmm_bstage<T, VEC, 2, 512>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
      } else {
        if (n_pad * 128 <= budget) rc = launch_spmm_bstage<T, VEC, 8>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
        else if (n_pad * 64 <= budget) rc = launch_spmm_bstage<T, VEC, 4>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
        else rc = launch_spmm_bstage<T, VEC, 2>(p, k, col_idx, vals, B, Y, alpha, beta, stream, dev, encode);
      }
      if (rc != B200SP_ERR_UNSUPPORTED) return rc;   // unsupported shape for the tensor map: fall through to the sliced kernel
    }
  }
  if (k % VEC == 0 && g_opt.spmm_sliced) {
    constexpr int KS = 8 * VEC, GROUPS = kSpmmThreads / 8;
    const int slices = (k + KS - 1) / KS;
    const int row_blocks = (int)((I.m + GROUPS - 1) / GROUPS);
    if ((long long)slices * row_blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
    int rc = launch(spmm_slice_kernel<T, VEC, kSpmmThreads>, dim3((unsigned)(slices * row_blocks)), dim3(kSpmmThreads), stream,
                    nullptr, 0, dev,
                    (int)I.m, k, row_blocks, p->row_ptr, col_idx, vals, B, Y, alpha, beta, kLongRow);
    if (rc != B200SP_OK || p->num_long == 0) return rc;
    return launch(spmm_long_row_kernel<T, VEC, kSpmmThreads>, dim3((unsigned)(slices * p->num_long)), dim3(kSpmmThreads), stream, nullptr, 0,
                  dev, k, p->num_long, (const int*)p->long_rows, p->row_ptr, col_idx, vals, B, Y, alpha, beta);
  }
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
              (int)nnz, row_ptr, col_idx, vals, x, y, alpha, beta, (const int*)sc->split_row, sc->carry, sc->tail);
  if (rc != B200SP_OK) return rc;
  if (tiles > 1)
    rc = launch(spmv_carry_fixup_kernel<T, kItems>, dim3((tiles + 127) / 128), dim3(128), stream, nullptr, 0, dev, tiles, row_ptr,
                (const int*)sc->split_row, (const float*)sc->carry, (const float*)sc->tail, y, alpha, beta);
  return rc;
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

int b200sp_probe_gather(const float* table, int64_t table_elems, int64_t gathers, float* sink, void* stream) {
  if (!table || !sink || table_elems <= 0 || (table_elems & (table_elems - 1)) != 0 || table_elems > ((int64_t)1 << 31) || gathers < 0)
    return B200SP_ERR_INVALID_ARG;
  DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != B200SP_OK) return rc;
  static int per_sm[64] = {};
  int d = 0;
  CU(cudaGetDevice(&d));
  if (!per_sm[d]) {
    CU(cudaFuncSetAttribute(probe_gather_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 0));
    int nb = 0;
    CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, probe_gather_kernel, 256, 0));
    per_sm[d] = nb > 0 ? nb : 1;
  }
  return launch(probe_gather_kernel, dim3((unsigned)(dev->sms * per_sm[d])), dim3(256), (cudaStream_t)stream, nullptr, 0, dev, table,
                (unsigned)(table_elems - 1), (long long)gathers, sink);
}

int64_t b200sp_noalloc_max_items(void) { return (int64_t)kNoAllocMaxTiles * kItems; }

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

int spmv_csc(int64_t m, int64_t n, int64_t nnz, const int32_t* col_ptr, const int32_t* row_idx, const void* vals, const void* x, void* y,
             float alpha, float beta, int dtype, void* stream) {
  return csc_call(false, m, n, nnz, 1, col_ptr, row_idx, vals, x, y, alpha, beta, dtype, stream);
}
int spmm_csc(int64_t m, int64_t n, int64_t nnz, int64_t k, const int32_t* col_ptr, const int32_t* row_idx, const void* vals, const void* B,
             void* Y, float alpha, float beta, int dtype, void* stream) {
  return csc_call(true, m, n, nnz, k, col_ptr, row_idx, vals, B, Y, alpha, beta, dtype, stream);
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

}  // extern "C"

template <typename T, int LPR, int VECW>
static int launch_ell_spmv(int64_t m, int width, const int32_t* col_ids, const T* vals, const T* x, T* y, float alpha, float beta,
                           cudaStream_t stream, DeviceInfo* dev) {
  constexpr int THREADS = 128;
  const long long blocks = (m * LPR + THREADS - 1) / THREADS;
  if (blocks >= (1LL << 31)) return B200SP_ERR_UNSUPPORTED;
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

extern "C" {

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

}  // extern "C"

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

extern "C" {

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
  char* base = nullptr;
  CU(cudaMallocAsync((void**)&base, bx + by + 256, stream));
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
  for (auto& kv : g_coo_cache) cudaFree(kv.second.row_ptr);
  g_coo_cache.clear();
  for (auto& kv : g_csc_cache) csc_free(kv.second);
  g_csc_cache.clear();
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
int64_t b200sp_launch_count(void) { return g_launches.load(); }

int b200sp_set_option(const char* name, int value) {
  if (!name) return B200SP_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!strcmp(name, "bstage_threads")) { if (value != 256 && value != 512 && value != 1024) return B200SP_ERR_INVALID_ARG; g_opt.bstage_threads = value; return B200SP_OK; }
  if (!strcmp(name, "bstage_nnz")) { if (value < 1024) return B200SP_ERR_INVALID_ARG; g_opt.bstage_nnz = value; return B200SP_OK; }
  if (!strcmp(name, "spmm_bstage")) { g_opt.spmm_bstage = value ? 1 : 0; return B200SP_OK; }
  if (!strcmp(name, "spmm_sliced")) { g_opt.spmm_sliced = value ? 1 : 0; return B200SP_OK; }
  if (!strcmp(name, "merge_threads")) { if (value != 64 && value != 128 && value != 256) return B200SP_ERR_INVALID_ARG; g_opt.merge_threads = value; return B200SP_OK; }
  if (!strcmp(name, "sub_lanes")) { if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8 && value != 16 && value != 32) return B200SP_ERR_INVALID_ARG; g_opt.sub_lanes = value; return B200SP_OK; }
  if (!strcmp(name, "merge_short")) { if (value != 8 && value != 16 && value != 32 && value != 64) return B200SP_ERR_INVALID_ARG; g_opt.merge_short = value; return B200SP_OK; }
  if (!strcmp(name, "merge_carve")) { if (value < -1 || value > 100) return B200SP_ERR_INVALID_ARG; g_opt.merge_carve = value; return B200SP_OK; }
  if (!strcmp(name, "merge_staged")) { g_opt.merge_staged = value ? 1 : 0; return B200SP_OK; }
  if (!strcmp(name, "merge_items")) { if (value != 1024 && value != 2048 && value != 4096) return B200SP_ERR_INVALID_ARG; g_opt.merge_items = value; return B200SP_OK; }
  if (!strcmp(name, "merge_stages")) { if (value < 2 || value > kMergeMaxStages) return B200SP_ERR_INVALID_ARG; g_opt.merge_stages = value; return B200SP_OK; }
  if (!strcmp(name, "merge_ctas")) { if (value < 1 || value > 8) return B200SP_ERR_INVALID_ARG; g_opt.merge_ctas = value; return B200SP_OK; }
  if (!strcmp(name, "uni_unroll")) { if (value != 1 && value != 2 && value != 4) return B200SP_ERR_INVALID_ARG; g_opt.uni_unroll = value; return B200SP_OK; }
  if (!strcmp(name, "uni_ctas")) { if (value < 0 || value > 32) return B200SP_ERR_INVALID_ARG; g_opt.uni_ctas = value; return B200SP_OK; }
  if (!strcmp(name, "spmv_kernel")) { if (value < -1 || value > 3) return B200SP_ERR_INVALID_ARG; g_opt.spmv_kernel = value; return B200SP_OK; }
  if (!strcmp(name, "x_l2_window")) { g_opt.x_l2_window = value ? 1 : 0; return B200SP_OK; }
  if (!strcmp(name, "row_stages")) { if (value < 2 || value > kRowMaxStages) return B200SP_ERR_INVALID_ARG; g_opt.row_stages = value; return B200SP_OK; }
  if (!strcmp(name, "row_smem_kb")) { if (value < 16 || value > 227) return B200SP_ERR_INVALID_ARG; g_opt.row_smem_kb = value; return B200SP_OK; }
  if (!strcmp(name, "row_threads")) { if (value != 128 && value != 256) return B200SP_ERR_INVALID_ARG; g_opt.row_threads = value; return B200SP_OK; }
  if (!strcmp(name, "row_ctas")) { if (value < 1 || value > 8) return B200SP_ERR_INVALID_ARG; g_opt.row_ctas = value; return B200SP_OK; }
  if (!strcmp(name, "row_unroll")) { if (value != 8 && value != 16) return B200SP_ERR_INVALID_ARG; g_opt.row_unroll = value; return B200SP_OK; }
  return B200SP_ERR_INVALID_ARG;
}

}  // extern "C"
