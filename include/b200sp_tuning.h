/*
 * b200sp -- tuning switches, test switches and measurement probes of libb200sp.so.
 *
 * Nothing here is needed to use the operations declared in b200sp.h (paper: Appendix C, Table 6, tasks 8-15); the
 * defaults are what the measurements kept with the library selected.  The switches exist so that each design choice
 * can be measured against its alternative on the same build, and so that failure paths can be reached in tests
 * without faulting a GPU.  Every accepted value of every switch is exercised against the CPU reference by the test
 * suite.  The probes have no counterpart in the paper: they measure the hardware rates that bound the kernels
 * (the paper's Appendix A sorts kernels by which such rate limits them).
 */
#ifndef B200SP_TUNING_H_
#define B200SP_TUNING_H_

#include "b200sp.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Sets a switch for the whole process; unknown names or values out of range return B200SP_ERR_INVALID_ARG.
 *  kernel choice
 *   "spmv_kernel"    -1 = choose from the plan statistics (default), 0 = merge-tile, 1 = row-direct, 2 = uniform-row,
 *                    3 = sub-warp per row; a kernel the matrix is not eligible for falls back to an eligible one
 *   "spmm_bstage"    1 = SpMM keeps a slice of B in shared memory when A has few columns (default), 0 = never
 *   "spmm_sliced"    1 = SpMM walks k in 128-byte slices so that a slice of B can stay in L2 (default), 0 = one pass
 *   "spmm_flat"      SpMM by chunks of 32 nonzeros per lane group instead of by rows (nnz-balanced, with carries between chunks and
 *                    tiles): 1 = always, 0 = never, 2 = when the rows are uneven (default: 5 % or more of the nonzeros in rows
 *                    longer than 128, a quarter or more of the rows empty, or a longest row far above the mean)
 *   "spmm_stage_a"   the k-sliced SpMM kernel's warps first copy their rows' (col, val) pairs into shared memory: 1 = yes, 0 = no,
 *                    2 = for BF16 storage only (default: measured 5-6 % faster there and 2-3 % slower for FP32)
 *   "spmm_ranges"    k-sliced SpMM on rows with ascending columns, one launch per column range so that the rows of B a
 *                    launch gathers from stay in L2: 1 = no ranges (default: measured slower, see the benchmarks' record),
 *                    0 = as many as make a range of B fit L2, 2, 3, 4 or 8 = that many
 *  merge-tile SpMV kernel
 *   "merge_items"    merge items per tile: 1024, 2048 (default) or 4096
 *   "merge_threads"  threads per CTA: 64, 128 (default) or 256
 *   "merge_carve"    shared-memory carveout in percent requested for it: 0, 25, 45 (default), 60, 75, 100 or -1 = leave to the driver
 *   "merge_short"    rows of up to this many products are added by one thread: 8, 16, 32 (default) or 64
 *   "merge_empty"    1 = when a quarter or more of the rows have no nonzeros the merge list holds only the other rows, and y
 *                    of the empty rows is written by a pass of its own, 0 = every row is a merge item (default: the list
 *                    measured 3 % slower on the power-law workload with 61 % empty rows)
 *  row-direct SpMV kernel
 *   "row_stages"     shared-memory stages per CTA, 2 (default) .. 4
 *   "row_ctas"       CTAs per SM the tiles are sized for, 1..4, default 3
 *   "row_smem_kb"    shared memory per SM it may use for stages: 48, 96, 160, 220 (default) or 227 (what is left stays L1)
 *   "row_threads"    threads per CTA, 128 or 256 (default)
 *   "row_unroll"     gathers in flight per thread, 8 (default) or 16
 *  other kernels
 *   "uni_unroll"     groups of four nonzeros in flight per thread of the uniform-row kernel: 1, 2 or 4; 0 (default) = 1
 *   "uni_ctas"       CTAs per SM for the uniform-row kernel: 1, 2, 4, 8 or 0 = as many as fit (default)
 *   "sub_lanes"      least number of lanes per row of the sub-warp kernel (1..32, power of two), 0 = from the mean row
 *                    length (default); more lanes are used where a lane would otherwise add more than 128 products
 *   "bstage_threads" threads per CTA of the SpMM kernel with B in shared memory: 256, 512 or 1024 (default)
 *   "bstage_nnz"     nonzeros of A per CTA that kernel aims for: 16384, 65536, 131072 or 524288; 0 (default) = chosen per
 *                    call so that the grid fills whole rounds of one CTA per SM ("bstage_quads" = 0: 131072)
 *   "bstage_stage_a" 1 = its warps first copy their rows' (col, val) pairs into shared-memory buffers of their own (default),
 *                    0 = the pairs are read from global memory inside the row loop
 *   "bstage_quads"   1 = that kernel runs on a copy of A made once per call (default): every row padded to whole groups of
 *                    four (16-bit offset, value) pairs and ordered so that neighbouring rows read different halves of a
 *                    shared-memory bank line, the rows taken in order of length (an order built once per plan, 8 m bytes);
 *                    a warp fetches its rows' groups with one bulk copy per array.  The copy takes about
 *                    (2 + bytes per value) * (nnz + 3 m) bytes from the library's pool for the duration of the call.
 *                    0 = the kernel walks the caller's col_idx / vals
 *   "x_l2_window"    1 = pin the gathered operand (x, or B for SpMM) in L2 with a per-launch access-policy window, 0 = off
 *                    (default; the measured effect is recorded with the benchmarks)
 *  launch
 *   "pdl"            1 = the SpMV and SpMM kernels are launched with programmatic stream serialisation (default): each begins
 *                    with griddepcontrol.wait, so it may be scheduled while the stream's previous kernel drains and touches no
 *                    memory before that kernel has completed; 0 = plain stream order
 *  memory
 *   "pool_keep_mb"   MiB of freed memory the library's pool keeps across synchronisation points, default 1024
 *                    (read when a device's pool is created, i.e. before the first call that allocates on it)
 *  logging
 *   "log"            1 = every plan that is built prints one line on stderr: row statistics, the SpMV kernel chosen, tiles and
 *                    scratch; 0 = silent (default).  B200SP_LOG=1 in the environment sets it when the library is loaded.
 *  test switches (they make a failure path run; none of them can fault or hang the device)
 *   "spin_limit"       polls after which a kernel's bounded wait on a shared-memory barrier gives up, default 1048576
 *   "debug_no_copies"  1 = the kernels that stage data through shared memory (row-direct SpMV, ELL row-direct SpMV, SpMM with
 *                      B in shared memory) issue no copy and arm no barrier, so their waits run out after "spin_limit" polls
 *                      with nothing in flight; the launch raises the flag that b200sp_check reports and its output is undefined
 *   "fail_alloc_after" N > 0: the N-th allocation the library makes from its memory pool from now on fails with
 *                      B200SP_ERR_ALLOC (the switch then clears itself); 0 = off (default)
 * "spmv_kernel", "merge_items" and "merge_empty" apply to plans created afterwards, the others to the next call. */
int b200sp_set_option(const char* name, int value);
/* Reads a switch back into *value (a host pointer).  Unknown names return B200SP_ERR_INVALID_ARG. */
int b200sp_get_option(const char* name, int* value);
/* Environment, read once when the library is loaded: B200SP_OPTIONS="name=value,name=value" sets switches as
 * b200sp_set_option would (an entry that is not accepted is reported on stderr and skipped); B200SP_LOG=1 sets "log". */

/* ---- measurement probes (no counterpart in the paper's operations) ----------------------------------------------
 * Each enqueues one kernel that does nothing but the access pattern named, so that the caller, timing it with events,
 * gets the hardware rate that bounds the corresponding library kernel.  All pointers are device pointers; `sink` is
 * one float that is (practically) never written.
 *
 * b200sp_probe_gather: `gathers` independent 4-byte reads of table[h(i) mod table_elems] (table_elems a power of two,
 *   h a hash computed in registers), eight in flight per thread, on as many CTAs as fit: the rate at which the SMs
 *   take random reads that miss L1, i.e. the bound on gathering x from a vector much larger than L1.
 * b200sp_probe_gather_ex: the same with entries of elem_bytes = 2 or 4 bytes and, with in_shared_memory = 1, with
 *   the table (at most 224 KB) first copied into each CTA's shared memory and gathered from there.
 * b200sp_probe_stream: reads `bytes` (a multiple of 16; buf 16-byte aligned) once with coalesced 128-bit loads: what
 *   a pure stream of the CSR arrays reaches at that size.
 * b200sp_probe_lines: `reads` random chunks of one, two or four consecutive 128-byte lines out of a buffer of `lines`
 *   lines (a power of two), each chunk by a group of group_lanes = 8, 16 or 32 lanes with 16 bytes per lane and
 *   in_flight = 4, 8 or 16 chunks in flight per group, into registers or, with to_shared_memory = 1 (group_lanes = 8
 *   only), into shared memory with cp.async: the L2-to-SM rate of SpMM's reads of B (the k-sliced kernel keeps four
 *   lines per group of eight lanes in registers).
 * b200sp_probe_spmv_gather: the gather phase of a CSR SpMV on the caller's arrays and nothing else: sum over all nonzeros
 *   of vals[p] * x[col_idx[p]] in per-thread partial sums (no rows, no y), one CTA of 1024 threads per SM, with
 *   unused_smem_kb (0 .. 200) KB of shared memory per SM carved out and left unused.  out receives one float per thread
 *   (SMs * 1024 floats; their sum is the sum above).  col_idx, vals 16-byte aligned; dtype as for spmv_csr; nnz is rounded
 *   down to a multiple of four.  It shows how the time of the gathers depends on the L1 that a kernel's shared memory leaves. */
int b200sp_probe_gather(const float* table, int64_t table_elems, int64_t gathers, float* sink, void* stream);
int b200sp_probe_gather_ex(const void* table, int64_t table_elems, int64_t gathers, int elem_bytes, int in_shared_memory, float* sink,
                           void* stream);
int b200sp_probe_stream(const void* buf, int64_t bytes, float* sink, void* stream);
int b200sp_probe_lines(const void* buf, int64_t lines, int64_t reads, int in_flight, int to_shared_memory, int group_lanes, float* sink,
                       void* stream);
int b200sp_probe_spmv_gather(int64_t nnz, const int32_t* col_idx, const void* vals, const void* x, int dtype, int unused_smem_kb, float* out,
                             void* stream);

#ifdef __cplusplus
}
#endif
#endif /* B200SP_TUNING_H_ */
