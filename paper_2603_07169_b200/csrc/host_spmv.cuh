// Host side of libb200sp.so: SpMV kernel selection and launches.
// One of the pieces of the single translation unit b200sp.cu; include/b200sp.h states the contract of every entry point.
#pragma once
#include "host_plan.cuh"
#include "spmv_kernels.cuh"
#include "spmv_row_kernels.cuh"
#include "spmv_uniform_kernels.cuh"
#include "probe_kernels.cuh"

namespace {

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
  tl_pdl_kernel = true;
  return launch_smem(kernel, dim3(grid), dim3(THREADS), smem, stream, x, (size_t)I.n * sizeof(T), dev, (int)I.m, (int)I.nnz,
                     p->row_ptr, col_idx, vals, x, y, alpha, beta, R, cap, tiles, stages, rot_lanes, dev->err_flag, 0, g_opt.spin_limit, g_opt.debug_no_copies);
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
  tl_pdl_kernel = true;
  return launch_smem(kernel, dim3(grid), dim3(THREADS), smem, stream, nullptr, 0, dev, (int)m, (int)(m * width), (const int*)nullptr, col_ids,
                     vals, x, y, alpha, beta, R, cap, tiles, stages, 0, dev->err_flag, width, g_opt.spin_limit, g_opt.debug_no_copies);
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
  tl_pdl_kernel = true;
  return launch(kernel, dim3((unsigned)blocks), dim3(THREADS), stream, x, (size_t)I.n * sizeof(T), dev, quads, col_idx, vals, x, y, alpha, beta);
}

template <typename T, int LPR>
int run_spmv_uniform_u(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                       cudaStream_t stream, DeviceInfo* dev) {
  const int unroll = g_opt.uni_unroll ? g_opt.uni_unroll : 1;   // one group: 32 registers, all 2048 threads of an SM resident (c2 FP32 65.5 us against 67 us with two groups, BF16 68.2 against 69.8 us)
  if (unroll == 1) return launch_uniform<T, LPR, 1>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (unroll == 4) return launch_uniform<T, LPR, 4>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
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

// y of the rows that are not in a merge list of non-empty rows: y = beta * y (zero when beta == 0).
template <typename T>
int run_empty_rows(b200sp_plan* p, T* y, float beta, cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  if (beta == 0.0f) return run_scale<T>(I.m, y, 0.0f, stream, dev);
  long long blocks = (I.m + 255) / 256;
  if (blocks > (long long)dev->sms * 16) blocks = (long long)dev->sms * 16;
  return launch(scale_empty_rows_kernel<T>, dim3((unsigned)blocks), dim3(256), stream, nullptr, 0, dev, (long long)I.m, p->row_ptr, y, beta);
}

template <typename T, int ITEMS, int SHORT = kShortMax>
int run_spmv_merge(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                   cudaStream_t stream, DeviceInfo* dev) {
  const b200sp_plan_info_t& I = p->info;
  const int tiles = I.spmv_tiles;
  const int rows = p->merge_compact ? p->compact_rows : (int)I.m;
  const int* rp = p->merge_compact ? p->compact_row_ptr : p->row_ptr;
  const int* rid = p->merge_compact ? p->compact_row_id : nullptr;
  int rc = B200SP_OK;
  if (rid) {
    rc = run_empty_rows<T>(p, y, beta, stream, dev);
    if (rc != B200SP_OK) return rc;
  }
#define B200SP_MERGE_LAUNCH(TH)                                                                                                          \
  {                                                                                                                                      \
    auto kernel = spmv_merge_tile_kernel<T, ITEMS, TH, SHORT>;                                                                           \
    if (g_opt.merge_carve >= 0) CU(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, g_opt.merge_carve));    \
    tl_pdl_kernel = true;                                                                                                                \
    rc = launch(kernel, dim3(tiles), dim3(TH), stream, x, (size_t)I.n * sizeof(T), dev, rows, (int)I.nnz, rp, col_idx, vals, x, y, alpha, \
                beta, (const int*)p->split_row, p->carry, p->tail, rid);                                                                 \
  }
  if (g_opt.merge_threads == 64) B200SP_MERGE_LAUNCH(64)
  else if (g_opt.merge_threads == 128) B200SP_MERGE_LAUNCH(128)
  else B200SP_MERGE_LAUNCH(256)
#undef B200SP_MERGE_LAUNCH
  if (rc != B200SP_OK) return rc;
  if (tiles > 1) {
    tl_pdl_kernel = true;
    rc = launch(spmv_carry_fixup_kernel<T, ITEMS>, dim3((tiles + 127) / 128), dim3(128), stream, nullptr, 0, dev, tiles, rp,
                (const int*)p->split_row, (const float*)p->carry, (const float*)p->tail, y, alpha, beta, rid);
  }
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
  tl_pdl_kernel = true;
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
  // no lane adds more than kSubwarpChain terms in sequence, whatever the mean says (the plan sends matrices with a row
  // longer than 32 * kSubwarpChain to the merge-tile kernel)
  while (lpr < 32 && ((long long)I.max_row_len + lpr - 1) / lpr > kSubwarpChain) lpr *= 2;
  switch (lpr) {
    case 1: return launch_subwarp<T, 1>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 2: return launch_subwarp<T, 2>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 4: return launch_subwarp<T, 4>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 8: return launch_subwarp<T, 8>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    case 16: return launch_subwarp<T, 16>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    default: return launch_subwarp<T, 32>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  }
}

// The merge-tile kernel by tile size and by the length up to which one thread adds a row.
template <typename T>
int run_spmv_merge_any(b200sp_plan* p, const int32_t* col_idx, const T* vals, const T* x, T* y, float alpha, float beta,
                       cudaStream_t stream, DeviceInfo* dev) {
  const int items = p->info.spmv_tile_items, sh = g_opt.merge_short;
#define B200SP_MERGE_BY_SHORT(FN, ITEMS)                                                      \
  if (sh == 8) return FN<T, ITEMS, 8>(p, col_idx, vals, x, y, alpha, beta, stream, dev);      \
  if (sh == 16) return FN<T, ITEMS, 16>(p, col_idx, vals, x, y, alpha, beta, stream, dev);    \
  if (sh == 64) return FN<T, ITEMS, 64>(p, col_idx, vals, x, y, alpha, beta, stream, dev);    \
  return FN<T, ITEMS, 32>(p, col_idx, vals, x, y, alpha, beta, stream, dev)
  if (items == 4096) return run_spmv_merge<T, 4096>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (items == 1024) return run_spmv_merge<T, 1024>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  B200SP_MERGE_BY_SHORT(run_spmv_merge, 2048);
#undef B200SP_MERGE_BY_SHORT
}

// The row-direct kernel gives its shared memory to stages and leaves little L1; that pays only when the gather of x is
// local (adjacent rows share lines).  The first call with a given col_idx samples that property (one small kernel, one
// synchronisation); matrices with scattered columns go to the merge-tile kernel instead.
int probe_col_locality(b200sp_plan* p, const int32_t* col_idx, cudaStream_t stream) {
  if (p->probed_col_idx == (const void*)col_idx) return B200SP_OK;
  const b200sp_plan_info_t& I = p->info;
  unsigned long long* d_out = p->probe_out;
  unsigned long long h[2] = {0, 0};
  if (!d_out) return B200SP_ERR_INVALID_ARG;
  cudaError_t e = cudaMemsetAsync(d_out, 0, sizeof h, stream);
  const int samples = I.m - 1 < 8192 ? (int)(I.m - 1) : 8192;
  if (e == cudaSuccess && samples > 0) {
    plan_col_locality_kernel<<<(samples + 127) / 128, 128, 0, stream>>>(p->row_ptr, col_idx, (int)I.m, samples, d_out);
    g_launches++;
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(h, d_out, sizeof h, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
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
      return run_spmv_merge_any<T>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
    }
  }
  if (I.spmv_kernel == 3) return run_spmv_subwarp<T>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (I.spmv_kernel == 2) return run_spmv_uniform<T>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  if (I.spmv_kernel == 1) return run_spmv_row_direct<T>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
  return run_spmv_merge_any<T>(p, col_idx, vals, x, y, alpha, beta, stream, dev);
}

}  // namespace
