// Host side of libb200sp.so: constants, tuning switches, device queries, the launch helper and argument checks.
// One of the pieces of the single translation unit b200sp.cu; include/b200sp.h states the contract of every entry point.
#pragma once
#include "../../include/b200sp_tuning.h"

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <tuple>
#include <vector>

#include "common.cuh"

using namespace b200sp;

namespace {

constexpr int kVersion = 200;  // 0.2.0

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
constexpr int kSpmmStageCap = 128;   // (col, val) pairs a warp of the k-sliced SpMM kernel can stage in shared memory
constexpr int kSmallNnz = 1 << 20;   // at or below this many nonzeros SpMV uses the sub-warp-per-row kernel
constexpr int kSubwarpChain = 128;   // longest sequential FP32 chain one lane of the sub-warp SpMV kernel may add
constexpr int kMediumRow = 128;   // SpMM: rows longer than this are added in blocks of this many products (second-to-last length bin)
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
  int uni_unroll = 0;     // groups of four nonzeros in flight per thread of the uniform-row kernel (1, 2 or 4); 0 = 1 (32 registers, full occupancy)
  int uni_ctas = 0;       // CTAs per SM for the uniform-row kernel (0 = as many as fit)
  int merge_items = 2048; // merge items per tile (1024, 2048 or 4096)
  int merge_threads = 128; // threads per CTA of the one-tile-per-CTA merge kernel (128 or 256)
  int bstage_threads = 1024; // threads per CTA of that kernel (256, 512 or 1024)
  int bstage_nnz = 0;        // nonzeros per CTA it aims for; 0 = chosen so that the grid fills whole rounds of one CTA per SM (the kernel on the caller's CSR arrays: 131072)
  int bstage_stage_a = 1;  // 1 = that kernel's warps copy their rows' (col, val) pairs into shared-memory buffers of their own (default), 0 = read them from global memory
  int bstage_quads = 1;    // 1 = that kernel runs on a copy of A re-laid once per call into padded quads ordered against bank conflicts (default), 0 = on the caller's CSR arrays
  int spmm_bstage = 1;     // 1 = hold the slice of B in shared memory when A has few columns (default), 0 = never
  int spmm_sliced = 1;     // 1 = k-sliced SpMM kernel (default), 0 = one pass over all of k
  int sub_lanes = 0;       // lanes per row of the sub-warp kernel (0 = from the mean row length)
  int merge_empty = 0;     // 1 = when a quarter or more of the rows have no nonzeros the merge list holds only the others, 0 = every row is a merge item (default: measured 3 % slower on the power-law workload, where the extra pass over y costs more than the skipped items save)
  int spmm_stage_a = 2;    // the k-sliced SpMM kernel's warps stage their rows' (col, val) pairs in shared memory: 1 = yes, 0 = no (broadcast loads from global memory), 2 = for BF16 storage only (default)
  int spmm_flat = 2;       // nnz-balanced SpMM kernel (a chunk of nonzeros per lane group instead of a row): 1 = always, 0 = never, 2 = when the rows are uneven (default)
  int spmm_ranges = 1;     // column ranges per slice of the k-sliced SpMM kernel with sorted columns: 1 = none (default), 0 = as many as make a range of B fit L2, 2, 3, 4, 8 = forced
  int merge_short = 32;    // rows up to this many products are added by one thread (8, 16, 32, 64)
  int pdl = 1;             // 1 = launch the kernels that begin with griddepcontrol.wait with programmatic stream serialisation
  int pool_keep_mb = 1024; // freed memory the library's pool keeps across synchronisation points, MiB (read when the pool is created)
  int merge_carve = 45;    // shared-memory carveout (percent) requested for it, -1 = leave to the driver
  int log = 0;                // 1 = one line on stderr per plan built: row statistics and the kernel chosen (also set by B200SP_LOG=1 in the environment)
  // test switches (failure paths that must be reachable without faulting a GPU)
  int spin_limit = 1 << 20;   // polls before a bounded barrier wait gives up
  int debug_no_copies = 0;    // 1 = the kernels that stage through shared memory issue no copy and arm no barrier: their waits run out
  int fail_alloc_after = 0;   // N > 0: the N-th allocation from the library's pool from now on fails (then the switch clears itself)
} g_opt;

struct DeviceInfo {
  bool known = false;
  int cc_major = 0, sms = 0, persist_max = 0, window_max = 0, l2_bytes = 0;
  size_t persist_set = 0;
  int* err_flag = nullptr;  // address of g_timeout_flag on this device: set by a kernel whose bounded wait ran out
  cudaMemPool_t pool = nullptr;  // the library's own stream-ordered pool: plan scratch and the host entry points' staging buffers
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

// The library's own memory pool on this device.  It keeps up to "pool_keep_mb" of freed memory across
// synchronisation points (the default pool of a device hands everything back at each of them, which makes
// every allocation of the next call map fresh memory); b200sp_cache_clear trims it to nothing.
int device_pool(DeviceInfo* d, cudaMemPool_t* out) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!d->pool) {
    int dev = 0;
    CU(cudaGetDevice(&dev));
    cudaMemPoolProps props = {};
    props.allocType = cudaMemAllocationTypePinned;
    props.handleTypes = cudaMemHandleTypeNone;
    props.location.type = cudaMemLocationTypeDevice;
    props.location.id = dev;
    cudaMemPool_t pool = nullptr;
    CU(cudaMemPoolCreate(&pool, &props));
    uint64_t keep = (uint64_t)(g_opt.pool_keep_mb < 0 ? 0 : g_opt.pool_keep_mb) << 20;
    cudaError_t e = cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
    if (e != cudaSuccess) { cudaMemPoolDestroy(pool); return cuda_fail(e, "cudaMemPoolSetAttribute"); }
    d->pool = pool;
  }
  *out = d->pool;
  return B200SP_OK;
}

int pool_alloc(DeviceInfo* d, void** ptr, size_t bytes, cudaStream_t stream) {
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_opt.fail_alloc_after > 0 && --g_opt.fail_alloc_after == 0) {   // injected failure (test switch)
      g_last_error = "out of device memory (injected)";
      return B200SP_ERR_ALLOC;
    }
  }
  cudaMemPool_t pool = nullptr;
  int rc = device_pool(d, &pool);
  if (rc != B200SP_OK) return rc;
  cudaError_t e = cudaMallocFromPoolAsync(ptr, bytes, pool, stream);
  if (e == cudaErrorMemoryAllocation) { (void)cudaGetLastError(); g_last_error = "out of device memory"; return B200SP_ERR_ALLOC; }
  if (e != cudaSuccess) return cuda_fail(e, "cudaMallocFromPoolAsync");
  return B200SP_OK;
}

// The flag that kernels with bounded waits raise: one int in the library image per device (zero when the module is
// loaded), so finding it neither allocates nor synchronises.
__device__ int g_timeout_flag;
int ensure_err_flag(DeviceInfo* d) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!d->err_flag) {
    void* ptr = nullptr;
    CU(cudaGetSymbolAddress(&ptr, g_timeout_flag));
    d->err_flag = static_cast<int*>(ptr);
  }
  return B200SP_OK;
}

thread_local bool tl_pdl_kernel = false;   // set by a launcher whose kernel begins with griddepcontrol.wait; consumed by the next launch

// Launch with an optional L2 access-policy window (persisting hits) over the gathered operand.
template <typename... KArgs, typename... Args>
int launch_smem(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, const void* win_ptr,
                size_t win_bytes, DeviceInfo* dev, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
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
  if (tl_pdl_kernel && g_opt.pdl) {
    // programmatic dependent launch: the kernel starts with griddepcontrol.wait, so it may be scheduled while the
    // previous kernel of the stream drains; nothing of it touches memory before that kernel has completed
    attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs++;
  }
  tl_pdl_kernel = false;
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
  void* block = nullptr;              // one allocation from the library's pool that holds every array below
  int32_t* split_row = nullptr;       // spmv tiles + 1
  float* carry = nullptr;             // spmv tiles
  float* tail = nullptr;              // spmv tiles
  int32_t* medium_rows = nullptr;     // rows of kMediumRow + 1 .. kLongRow nonzeros, ascending
  int32_t* long_rows = nullptr;       // rows longer than kLongRow, ascending
  unsigned long long* probe_out = nullptr;  // two counters for the column-locality probe
  int num_medium = 0, num_long = 0;
  const void* probed_col_idx = nullptr;   // col_idx the column-locality probe last ran on
  int32_t* flat_tile_row = nullptr;       // tile starts of the nnz-balanced SpMM kernel (a pool block of its own, built on first use)
  // merge list over the rows that have nonzeros (matrices with many empty rows)
  void* compact_block = nullptr;          // one pool block: row ids, their offsets, block counts
  int compact_rows = 0;                   // number of rows that have nonzeros (0 = the list has not been built)
  bool merge_compact = false;             // the SpMV merge list (split_row) was built over that list
  int32_t* compact_row_id = nullptr;      // compact_rows matrix row numbers, ascending
  int32_t* compact_row_ptr = nullptr;     // compact_rows + 1 offsets
  // column ranges of the k-sliced SpMM kernel (rows with ascending columns): built on the first SpMM call with a given col_idx
  void* cuts_block = nullptr;             // (ranges - 1) * m cut positions, a pool block of its own
  const void* cuts_col_idx = nullptr;     // col_idx they were computed from
  int cuts_ranges = 0;                    // number of ranges they describe (0 = none computed)
  bool cols_sorted = false;               // every row's columns ascend
  // processing order of the SpMM kernel with B in shared memory: rows of at most kLongRow nonzeros sorted by length, in blocks of quad_gpw
  void* quad_block = nullptr;             // one pool block: row numbers, row lengths, block offsets (built on first use)
  int32_t* quad_row = nullptr;            // quad_blocks * quad_gpw row numbers (-1 = unused slot)
  int32_t* quad_len = nullptr;            // their lengths
  int32_t* quad_pos = nullptr;            // quad_blocks + 1: where each block's quads start in the per-call copy of A
  int quad_gpw = 0, quad_blocks = 0;
  const void* probed_key = nullptr;       // host entry points: the HOST col_idx that verdict belongs to
  bool cols_local = true;                 // its verdict: adjacent rows share most of their lines of x
};
