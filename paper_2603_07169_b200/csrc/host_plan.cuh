// Host side of libb200sp.so: the plan pass (row statistics, bins, splits, medium- and long-row lists) and the plan cache.
// One of the pieces of the single translation unit b200sp.cu; include/b200sp.h states the contract of every entry point.
#pragma once
#include "host_runtime.cuh"
#include "plan_kernels.cuh"

namespace {

// Plans cached by the one-shot entry points, keyed on (device, row_ptr address, m, n, nnz).  The address may be a device
// pointer (spmv_csr, spmm_csr) or a host pointer (spmv_csr_host, spmm_csr_host); the two never collide in a unified
// address space.  At most kCacheCap plans are kept: the least recently used one is dropped when another is added.
typedef std::tuple<int, const void*, int64_t, int64_t, int64_t> PlanKey;
struct CachedPlan { b200sp_plan* plan = nullptr; uint64_t stamp = 0; };
std::map<PlanKey, CachedPlan> g_cache;
uint64_t g_cache_clock = 0;
constexpr size_t kCacheCap = 1024;

// Frees a plan.  With stream_ordered the block goes back to the pool in the order of `stream` (the caller
// knows that every kernel that used the plan ran there); otherwise the device is synchronised first.
int plan_free(b200sp_plan* p, bool stream_ordered = false, cudaStream_t stream = nullptr) {
  if (!p) return B200SP_OK;
  int rc = B200SP_OK;
  if (p->block || p->cuts_block || p->compact_block || p->flat_tile_row || p->quad_block) {
    cudaError_t e = cudaSuccess;
    if (stream_ordered) {
      if (p->block) e = cudaFreeAsync(p->block, stream);
      if (p->cuts_block && e == cudaSuccess) e = cudaFreeAsync(p->cuts_block, stream);
      if (p->compact_block && e == cudaSuccess) e = cudaFreeAsync(p->compact_block, stream);
      if (p->flat_tile_row && e == cudaSuccess) e = cudaFreeAsync(p->flat_tile_row, stream);
      if (p->quad_block && e == cudaSuccess) e = cudaFreeAsync(p->quad_block, stream);
    } else {
      int cur = 0;
      e = cudaGetDevice(&cur);
      if (e == cudaSuccess && cur != p->device) e = cudaSetDevice(p->device);
      if (e == cudaSuccess) e = cudaDeviceSynchronize();
      if (e == cudaSuccess && p->block) e = cudaFree(p->block);
      if (e == cudaSuccess && p->cuts_block) e = cudaFree(p->cuts_block);
      if (e == cudaSuccess && p->compact_block) e = cudaFree(p->compact_block);
      if (e == cudaSuccess && p->flat_tile_row) e = cudaFree(p->flat_tile_row);
      if (e == cudaSuccess && p->quad_block) e = cudaFree(p->quad_block);
      if (cur != p->device) cudaSetDevice(cur);
    }
    if (e != cudaSuccess) rc = cuda_fail(e, "freeing a plan");
  }
  delete p;
  return rc;
}

// The list of the rows that have nonzeros (their numbers and their offsets), built on the device in stream order and kept with
// the plan: used by the merge-tile SpMV kernel under the switch "merge_empty" and by the nnz-balanced SpMM kernel.  Needs
// info.bin_rows[0] (the number of empty rows).  No synchronisation.
int plan_compact_rows(b200sp_plan* p, cudaStream_t stream, DeviceInfo* dev) {
  if (p->compact_block) return B200SP_OK;
  b200sp_plan_info_t& I = p->info;
  const int64_t m = I.m, mc = m - I.bin_rows[0];
  auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
  const int blocks = (int)((m + kCompactBlock - 1) / kCompactBlock);
  const size_t o_id = 0, o_rp = o_id + up((size_t)(mc + 1) * 4), o_bc = o_rp + up((size_t)(mc + 1) * 4), total = o_bc + up((size_t)(blocks + 1) * 4);
  void* blk = nullptr;
  int rc = pool_alloc(dev, &blk, total, stream);
  if (rc != B200SP_OK) return rc;
  char* b2 = (char*)blk;
  int32_t* row_id = (int32_t*)(b2 + o_id);
  int32_t* row_ptr_c = (int32_t*)(b2 + o_rp);
  int* d_bc = (int*)(b2 + o_bc);
  plan_compact_count_kernel<<<blocks, 256, 0, stream>>>(p->row_ptr, (int)m, d_bc);
  plan_compact_scan_kernel<<<1, 1024, 0, stream>>>(d_bc, blocks);
  plan_compact_write_kernel<<<blocks, 256, 0, stream>>>(p->row_ptr, (int)m, (int)I.nnz, d_bc, row_id, row_ptr_c);
  g_launches += 3;
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { cudaFreeAsync(blk, stream); return cuda_fail(e, "list of non-empty rows"); }
  p->compact_block = blk;
  p->compact_row_id = row_id;
  p->compact_row_ptr = row_ptr_c;
  p->compact_rows = (int)mc;
  I.scratch_bytes += (int64_t)total;
  return B200SP_OK;
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
  const int items = g_opt.merge_items;
  I.spmv_tile_items = items;
  I.spmv_tiles = (int32_t)((m + nnz + items - 1) / items);
  I.spmv_kernel = g_opt.spmv_kernel >= 0 ? g_opt.spmv_kernel : 0;
  if (m == 0) { *out = p; return B200SP_OK; }

  // one block from the pool: statistics, counters, split points, carries, tails, medium- and long-row lists
  const size_t nt = (size_t)I.spmv_tiles;
  const size_t long_cap = (size_t)(nnz / (kLongRow + 1)) + 1;     // rows longer than kLongRow: at most this many
  const size_t mid_cap = (size_t)(nnz / (kMediumRow + 1)) + 1;    // rows longer than kMediumRow
  auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
  const size_t o_stats = 0, o_count = o_stats + up(sizeof(PlanStats)), o_split = o_count + 256, o_carry = o_split + up((nt + 1) * 4),
               o_tail = o_carry + up((nt + 1) * 4), o_mid = o_tail + up((nt + 1) * 4), o_long = o_mid + up(mid_cap * 4),
               total = o_long + up(long_cap * 4);
  PlanStats h = {};
  h.min_len = 0x7FFFFFFF;
  auto fail = [&](int code) { plan_free(p, true, stream); cudaStreamSynchronize(stream); return code; };
#define CUP(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(cuda_fail(e_, #call)); } while (0)
  rc = pool_alloc(dev, &p->block, total, stream);
  if (rc != B200SP_OK) { delete p; return rc; }
  char* base = (char*)p->block;
  PlanStats* d_stats = (PlanStats*)(base + o_stats);
  int* d_count = (int*)(base + o_count);                       // two list counters
  p->probe_out = (unsigned long long*)(base + o_count + 16);   // two probe counters
  p->split_row = (int32_t*)(base + o_split);
  p->carry = (float*)(base + o_carry);
  p->tail = (float*)(base + o_tail);
  p->medium_rows = (int32_t*)(base + o_mid);
  p->long_rows = (int32_t*)(base + o_long);
  I.scratch_bytes = (int64_t)total;
  CUP(cudaMemcpyAsync(d_stats, &h, sizeof h, cudaMemcpyHostToDevice, stream));
  {
    const int blocks = (int)((m + 256 * 8 - 1) / (256 * 8));
    const int grid = blocks < dev->sms * 8 ? (blocks > 0 ? blocks : 1) : dev->sms * 8;
    plan_stats_kernel<<<grid, 256, 0, stream>>>(row_ptr, (int)m, d_stats);
    g_launches++;
  }
  plan_merge_split_kernel<<<(unsigned)((nt + 1 + 255) / 256), 256, 0, stream>>>(row_ptr, (int)m, (int)nnz, items, (int)nt, p->split_row);
  g_launches++;
  CUP(cudaGetLastError());
  CUP(cudaMemcpyAsync(&h, d_stats, sizeof h, cudaMemcpyDeviceToHost, stream));
  CUP(cudaStreamSynchronize(stream));
  if (!h.bad && h.bin_rows[4] + h.bin_rows[5] > 0) {   // lists of the rows in the last two length bins, sorted on the host
    const size_t n_mid = (size_t)h.bin_rows[4], n_long = (size_t)h.bin_rows[5];
    if (n_mid > mid_cap || n_long > long_cap) return fail(B200SP_ERR_BAD_CSR);   // cannot happen for a monotone row_ptr
    CUP(cudaMemsetAsync(d_count, 0, 2 * sizeof(int), stream));
    const int blocks = (int)((m + 255) / 256);
    plan_row_lists_kernel<<<blocks < dev->sms * 8 ? blocks : dev->sms * 8, 256, 0, stream>>>(
        row_ptr, (int)m, kMediumRow, kLongRow, (int)n_mid, (int)n_long, p->medium_rows, p->long_rows, d_count);
    g_launches++;
    CUP(cudaGetLastError());
    std::vector<int32_t> tmp(n_mid + n_long);
    if (n_mid) CUP(cudaMemcpyAsync(tmp.data(), p->medium_rows, n_mid * sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    if (n_long) CUP(cudaMemcpyAsync(tmp.data() + n_mid, p->long_rows, n_long * sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    CUP(cudaStreamSynchronize(stream));
    std::sort(tmp.begin(), tmp.begin() + n_mid);
    std::sort(tmp.begin() + n_mid, tmp.end());
    if (n_mid) CUP(cudaMemcpyAsync(p->medium_rows, tmp.data(), n_mid * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    if (n_long) CUP(cudaMemcpyAsync(p->long_rows, tmp.data() + n_mid, n_long * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    CUP(cudaStreamSynchronize(stream));
    p->num_medium = (int)n_mid;
    p->num_long = (int)n_long;
  }
  // Many rows without nonzeros (a quarter or more): the merge list is built over the rows that have nonzeros only, and the
  // split points are searched again over that list.
  if (!h.bad && g_opt.merge_empty && nnz > 0 && (int64_t)h.bin_rows[0] * 4 >= m) {
    for (int j = 0; j < B200SP_NUM_BINS; ++j) I.bin_rows[j] = (int64_t)h.bin_rows[j];
    rc = plan_compact_rows(p, stream, dev);
    if (rc != B200SP_OK) return fail(rc);
    const int64_t mc = p->compact_rows;
    const size_t ntc = (size_t)((mc + nnz + items - 1) / items);     // fewer items, fewer tiles: the arrays sized above suffice
    plan_merge_split_kernel<<<(unsigned)((ntc + 1 + 255) / 256), 256, 0, stream>>>(p->compact_row_ptr, (int)mc, (int)nnz, items, (int)ntc, p->split_row);
    g_launches++;
    CUP(cudaGetLastError());
    CUP(cudaStreamSynchronize(stream));
    p->merge_compact = true;
    I.spmv_tiles = (int32_t)ntc;
  }
#undef CUP
  if (h.bad) { plan_free(p, true, stream); cudaStreamSynchronize(stream); return B200SP_ERR_BAD_CSR; }
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
  if (nnz > 0 && nnz <= kSmallNnz && h.max_len <= 32 * kSubwarpChain && !uniform_ok && !(row_direct_ok && m >= (int64_t)kRowThreads * dev->sms)) choice = 3;
  if (g_opt.spmv_kernel == 3) choice = h.max_len <= 32 * kSubwarpChain ? 3 : 0;
  if (g_opt.spmv_kernel == 0) choice = 0;
  if (g_opt.spmv_kernel == 1) choice = row_direct_possible ? 1 : 0;
  if (g_opt.spmv_kernel == 2) choice = uniform_ok ? 2 : (row_direct_ok ? 1 : 0);
  I.spmv_kernel = choice;
  if (g_opt.log) {
    static const char* const kname[4] = {"merge-tile", "row-direct", "uniform-row", "sub-warp"};
    fprintf(stderr, "b200sp plan: m=%lld n=%lld nnz=%lld rows by length 0|1-4|5-32|33-128|129-1024|>1024 = %lld|%lld|%lld|%lld|%lld|%lld min=%d max=%d "
                    "spmv kernel=%s tiles=%d x %d items%s scratch=%lld bytes\n",
            (long long)m, (long long)n, (long long)nnz, (long long)I.bin_rows[0], (long long)I.bin_rows[1], (long long)I.bin_rows[2], (long long)I.bin_rows[3],
            (long long)I.bin_rows[4], (long long)I.bin_rows[5], I.min_row_len, I.max_row_len, kname[choice & 3], I.spmv_tiles, I.spmv_tile_items,
            p->merge_compact ? " (non-empty rows only)" : "", (long long)I.scratch_bytes);
  }
  *out = p;
  return B200SP_OK;
}

int check_common(const b200sp_plan* p, const void* col_idx, const void* vals, const void* dense_in, const void* dense_out, int dtype) {
  if (!p) return B200SP_ERR_INVALID_ARG;
  if (dtype != B200SP_F32 && dtype != B200SP_BF16) return B200SP_ERR_INVALID_ARG;
  const b200sp_plan_info_t& I = p->info;
  if (I.nnz > 0 && (!col_idx || !vals || !dense_in)) return B200SP_ERR_INVALID_ARG;
  if (I.m > 0 && !dense_out) return B200SP_ERR_INVALID_ARG;
  if (!aligned16(col_idx) || !aligned16(vals) || !aligned16(dense_in) || !aligned16(dense_out)) return B200SP_ERR_INVALID_ARG;
  int cur = 0;
  CU(cudaGetDevice(&cur));
  if (I.m > 0 && cur != p->device) return B200SP_ERR_INVALID_ARG;   // a plan belongs to the device it was created on
  return B200SP_OK;
}

// Looks `key` up; a hit refreshes its stamp.  The caller holds no lock.
b200sp_plan* cache_find(const PlanKey& key) {
  std::lock_guard<std::mutex> lock(g_mutex);
  auto it = g_cache.find(key);
  if (it == g_cache.end()) return nullptr;
  it->second.stamp = ++g_cache_clock;
  return it->second.plan;
}

// Adds a plan under `key` (or returns the one another thread added first) and drops the least recently used
// plan beyond the cap.  Dropping synchronises the device of the dropped plan.
b200sp_plan* cache_insert(const PlanKey& key, b200sp_plan* p) {
  b200sp_plan* victim = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    auto ins = g_cache.emplace(key, CachedPlan{p, ++g_cache_clock});
    if (!ins.second) { victim = p; p = ins.first->second.plan; }
    else if (g_cache.size() > kCacheCap) {
      auto oldest = g_cache.end();
      for (auto it = g_cache.begin(); it != g_cache.end(); ++it)
        if (it->second.plan != p && (oldest == g_cache.end() || it->second.stamp < oldest->second.stamp)) oldest = it;
      if (oldest != g_cache.end()) { victim = oldest->second.plan; g_cache.erase(oldest); }
    }
  }
  if (victim) plan_free(victim);
  return p;
}

int get_cached_plan(b200sp_plan** out, int64_t m, int64_t n, int64_t nnz, const int32_t* row_ptr, cudaStream_t stream) {
  int dev = 0;
  CU(cudaGetDevice(&dev));
  const PlanKey key = std::make_tuple(dev, (const void*)row_ptr, m, n, nnz);
  if (b200sp_plan* hit = cache_find(key)) { *out = hit; return B200SP_OK; }
  b200sp_plan* p = nullptr;
  int rc = b200sp_plan_create(&p, m, n, nnz, row_ptr, stream);
  if (rc != B200SP_OK) return rc;
  *out = cache_insert(key, p);
  return B200SP_OK;
}

}  // namespace
