#!/usr/bin/env python
"""Benchmark of the CSR SpMV / SpMM hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras]
    python bench.py --probes          the hardware rates behind the secondary bounds (gather, stream, full-line reads)
    python bench.py --paper-sweep     the paper's own SpMV / SpMM sizes, speed-up over a naive kernel and its score P

Headline (one JSON line on stdout): effective HBM GB/s of CSR SpMV on the uniform 16-nonzeros-per-row
workload (m = n = 2^20, FP32, alpha 1.5, beta 0.5), i.e. algorithmic bytes per call divided by the
device time per call, through the C ABI (spmv_csr) with a cached plan.  One "step" is one spmv_csr
call; on this workload (equal rows) that is one launch of the uniform-row kernel.  Inputs are resident
in HBM; to keep every call cold, the steps rotate over R independent device copies of all operands whose
total size is several times the L2 capacity, so no flush sits inside the timed region.  The same line carries the
roofline fraction against the measured copy bandwidth, an end-to-end figure through spmv_csr_host
(host buffers, copies inside the timed region), the CPU oracle timed on the host cores, the other
workloads (BF16, R-MAT, 27-point stencil, SpMM) as extras, and the SM clocks sampled while running.

With --gpus N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its
own GPU: the path is single-GPU by design, there is no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "SpMV/SpMM effective HBM GB/s (fraction of B200 peak); GFLOP/s at 2*nnz*k"
FALLBACK_HBM_GBS = 6650.0

def ncu_record(workload: str, dtype: str):
    """What one ncu capture of the dominant kernel of (workload, dtype) measured, per launch: profiles/traffic.json, written
    from ncu's CSV by `python -m paper_2603_07169_b200.ncu_summary` (None if there is no capture)."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        return json.load(f).get("%s_%s" % (workload, dtype))


def ncu_traffic(workload: str, dtype: str):
    rec = ncu_record(workload, dtype)
    return None if rec is None else rec.get("dram_bytes")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) from a background thread."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.samples = []
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # pragma: no cover
            self.err = repr(e)

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                clk = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.perf_counter(), clk, reasons))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.ok:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()

    def summary(self, t0: float, t1: float):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable"]}
        sel = [s for s in self.samples if t0 <= s[0] <= t1]
        inside = len(sel)
        if not sel:                      # a region shorter than the sampling period: the two samples that bracket it, and say so
            before = [s for s in self.samples if s[0] < t0][-1:]
            after = [s for s in self.samples if s[0] > t1][:1]
            sel = before + after
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
                 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}
        seen = 0
        for s in sel:
            seen |= s[2]
        reasons = [n for bit, n in names.items() if seen & bit]
        clk = sorted(s[1] for s in sel)
        return {"sm_mhz": clk[len(clk) // 2] if clk else None, "sm_max_mhz": self.max_sm, "reasons": reasons,
                "samples": inside, "bracketing_samples": len(sel) - inside if not inside else 0}


# ------------------------------------------------------------------------------------------ helpers
def stored(a, dtype):
    import gen
    if a is None:
        return None
    return gen.to_bf16(a) if dtype == "bf16" else np.ascontiguousarray(a, np.float32)


def up(a, dev):
    import torch
    return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).to(dev)


class DeviceSet:
    """One device copy of all operands of a workload."""

    def __init__(self, w, dtype, dev):
        import torch
        A = w.A
        self.rp, self.ci = up(A.row_ptr, dev), up(A.col_idx, dev)
        self.va = up(stored(A.vals, dtype), dev)
        dense = w.B if w.k else w.x
        self.inp = up(stored(dense, dtype), dev)
        kk = max(w.k, 1)
        if w.beta != 0 and w.y0 is not None:
            self.out = up(stored(w.y0, dtype), dev)
        else:
            self.out = torch.zeros(A.m * kk, dtype=torch.float32 if dtype == "f32" else torch.int16, device=dev)


def measure(w, dtype, steps, warmup, dev, l2_bytes, barrier=None, min_copies=2, max_bytes=8 << 30, cusparse=None):
    """Times `steps` calls back to back with one CUDA-event pair on the launching stream; the calls rotate
    over R device copies of all operands (R * bytes >= 4 * L2).  Returns a dict of figures."""
    import torch
    import gen
    import paper_2603_07169_b200 as b200sp
    A = w.A
    e = 4 if dtype == "f32" else 2
    abytes = gen.algorithmic_bytes(A.m, A.n, A.nnz, e, w.beta, w.k)
    R = max(min_copies, -(-4 * l2_bytes // abytes))
    R = max(1, min(R, max_bytes // max(abytes, 1), 256))
    sets = [DeviceSet(w, dtype, dev) for _ in range(R)]
    stream = torch.cuda.current_stream()

    def call(s, st=stream):                  # st: the launching stream (a capture stream when recorded into a CUDA graph)
        if w.k:
            b200sp.spmm_csr(A.m, A.n, A.nnz, w.k, s.rp, s.ci, s.va, s.inp, s.out, w.alpha, w.beta, dtype, st)
        else:
            b200sp.spmv_csr(A.m, A.n, A.nnz, s.rp, s.ci, s.va, s.inp, s.out, w.alpha, w.beta, dtype, st)

    t_plan0 = time.perf_counter()
    call(sets[0])                       # first call builds and caches the plan for this row_ptr
    torch.cuda.synchronize()
    plan_ms = (time.perf_counter() - t_plan0) * 1e3
    for s in sets[1:]:
        call(s)
    for i in range(max(warmup, 3)):
        call(sets[i % R])
    torch.cuda.synchronize()
    if barrier:
        barrier()
    l0 = b200sp.b200sp_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    ev0.record(stream)
    for i in range(steps):
        call(sets[i % R])
    ev1.record(stream)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    if barrier:
        barrier()
    ms = ev0.elapsed_time(ev1)
    launches = b200sp.b200sp_launch_count() - l0
    # isolated single calls (event pair around each, cold L2 by rotation): median
    iso = []
    for i in range(min(steps, 50)):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        call(sets[i % R])
        b.record(stream)
        b.synchronize()
        iso.append(a.elapsed_time(b))
    iso.sort()
    # warm: the same operand set back to back (whatever fits stays in L2; not comparable with the HBM roofline)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    call(sets[0])
    a.record(stream)
    for i in range(min(steps, 50)):
        call(sets[0])
    b.record(stream)
    b.synchronize()
    warm_ms = a.elapsed_time(b) / min(steps, 50)
    ms_step = ms / steps
    flops = 2.0 * A.nnz * max(w.k, 1)
    res = {"ms_total": ms, "ms_per_step": ms_step, "ms_per_step_isolated_median": iso[len(iso) // 2], "ms_per_step_warm": warm_ms,
           "gbs": abytes / ms_step * 1e-6,
           "gflops": flops / ms_step * 1e-6, "algorithmic_bytes": abytes, "copies": R, "launches": launches,
           "plan_ms_first_call": plan_ms, "t0": t0, "t1": t1, "nnz": A.nnz, "m": A.m}
    res["cusparse_ms"] = None
    if cusparse is not None:
        try:
            res["cusparse_ms"] = cusparse.time(sets, w, dtype, min(steps, 20), stream)
        except Exception as ex:  # pragma: no cover
            res["cusparse_ms"] = "unavailable: %r" % (ex,)
    res["_sets"] = sets
    res["_call"] = call
    return res


def measure_format(kind, w, dtype, steps, dev, l2_bytes):
    """COO / ELL / CSC front ends on a CSR workload converted on the host (same rotation protocol as `measure`).
    Algorithmic bytes: COO as CSR (the row offsets derived from row_indices are cached); ELL m*width*(4+e) + n*e + m*e (+ m*e)."""
    import torch
    import gen
    import paper_2603_07169_b200 as b200sp
    A = w.A
    e = 4 if dtype == "f32" else 2
    ywrite = A.m * e * (2 if w.beta != 0 else 1)
    if kind == "coo":
        r, c, v = gen.csr_to_coo(A)
        arrays = (r, c, stored(v, dtype))
        # row_indices are read once, when the row offsets are derived and cached; per call the traffic is that of CSR
        abytes = A.nnz * (4 + e) + (A.m + 1) * 4 + A.n * e + ywrite
    elif kind == "csc":
        cp, ri, v = gen.csr_to_csc(A)
        arrays = (cp, ri, stored(v, dtype))
        abytes = A.nnz * (4 + e) + (A.n + 1) * 4 + A.n * e + ywrite      # the CSC arrays once, x, y
    else:
        W, ci, va = gen.csr_to_ell(A)
        arrays = (ci, stored(va, dtype))
        abytes = A.m * W * (4 + e) + A.n * e + ywrite
    R = int(max(2, min(64, -(-4 * l2_bytes // abytes))))
    if kind == "csc":
        R = 2        # every cached CSC pattern holds 12 bytes + a value per nonzero of plan memory
    x_s = stored(w.x, dtype)
    sets = []
    for _ in range(R):
        out = up(stored(w.y0, dtype), dev) if (w.beta != 0 and w.y0 is not None) else torch.zeros(A.m, dtype=torch.float32 if dtype == "f32" else torch.int16, device=dev)
        sets.append([up(a, dev) for a in arrays] + [up(x_s, dev), out])
    stream = torch.cuda.current_stream()
    if kind == "coo":
        call = lambda s: b200sp.spmv_coo(A.m, A.n, A.nnz, s[0], s[1], s[2], s[3], s[4], w.alpha, w.beta, dtype, stream)
    elif kind == "csc":
        call = lambda s: b200sp.spmv_csc(A.m, A.n, A.nnz, s[0], s[1], s[2], s[3], s[4], w.alpha, w.beta, dtype, stream)
    else:
        call = lambda s: b200sp.spmv_ell(A.m, A.n, W, s[0], s[1], s[2], s[3], w.alpha, w.beta, dtype, stream)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    call(sets[0])                       # first call: whatever the front end derives from the pattern (row offsets, transpose plan)
    torch.cuda.synchronize()
    first_ms = (time.perf_counter() - t0) * 1e3
    for s_ in sets[1:]:
        call(s_)
    for i in range(5):
        call(sets[i % R])
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for i in range(steps):
        call(sets[i % R])
    b.record(stream)
    b.synchronize()
    ms = a.elapsed_time(b) / steps
    b200sp.b200sp_cache_clear()
    return {"ms_per_step": round(ms, 5), "gbs": round(abytes / ms * 1e-6, 1), "algorithmic_bytes": abytes, "copies": R,
            "first_call_ms": round(first_ms, 3)}


def latency_floor(call, sets, dev, nbytes):
    """Per-call device time of 100 calls replayed from a CUDA graph, beside an empty kernel and a copy of the same bytes."""
    import torch
    import paper_2603_07169_b200 as b200sp

    def graph_us(fn, calls=100, replays=5):
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(calls):
                    fn(i)
        torch.cuda.current_stream().wait_stream(side)
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(replays):
            g.replay()
        b.record()
        b.synchronize()
        return a.elapsed_time(b) / (replays * calls) * 1e3

    out = {}
    try:
        tab = torch.zeros(1024, dtype=torch.float32, device=dev)
        sink = torch.zeros(1, dtype=torch.float32, device=dev)
        src = torch.zeros(nbytes // 8, dtype=torch.float32, device=dev)
        dst = torch.empty_like(src)
        out["graph_replay_us_per_call"] = round(graph_us(lambda i: call(sets[i % len(sets)], torch.cuda.current_stream())), 3)
        out["empty_kernel_us"] = round(graph_us(lambda i: b200sp.b200sp_probe_gather(tab, 1024, 0, sink, torch.cuda.current_stream())), 3)
        out["copy_same_bytes_us"] = round(graph_us(lambda i: dst.copy_(src)), 3)
        # the same copy over as many independent buffers as the SpMV calls rotate over, so that it too reads cold lines
        srcs = [torch.zeros(nbytes // 8, dtype=torch.float32, device=dev) for _ in range(len(sets))]
        out["copy_same_bytes_cold_us"] = round(graph_us(lambda i: dst.copy_(srcs[i % len(srcs)])), 3)
    except Exception as ex:  # pragma: no cover
        out["latency_floor_error"] = repr(ex)
    return out


def aggregate_over_ranks(ms_local: float, bytes_per_step: int, steps: int, world: int, dist=None, device="cpu"):
    """Whole-job figures for N independent replicas: time = max over ranks, work = sum over ranks.
    Returns (ms_per_step, GB/s).  With world == 1 nothing is communicated."""
    ms = ms_local
    if world > 1:
        import torch
        t = torch.tensor([ms_local], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    ms_step = ms / steps
    return ms_step, world * bytes_per_step / ms_step * 1e-6


def probe_gather_rate(n_elems: int, dev) -> float:
    """Random 4-byte gathers per second from a table of n_elems floats (rounded up to a power of two), L1-missing."""
    import torch
    import paper_2603_07169_b200 as b200sp
    T = 1 << max(10, (n_elems - 1).bit_length())
    table = torch.zeros(T, dtype=torch.float32, device=dev)
    sink = torch.zeros(1, dtype=torch.float32, device=dev)
    gathers = 1 << 26
    stream = torch.cuda.current_stream()
    for _ in range(3):
        b200sp.b200sp_probe_gather(table, T, gathers, sink, stream)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(5):
        b200sp.b200sp_probe_gather(table, T, gathers, sink, stream)
    b.record(stream)
    b.synchronize()
    return 5 * gathers / (a.elapsed_time(b) * 1e-3)


def probe_gather_phase(w, dtype, dev, l2_bytes) -> float:
    """Seconds the gather phase of SpMV alone takes on this workload's own matrix (b200sp_probe_spmv_gather, no shared memory
    carved out), each repetition started cold (a buffer larger than L2 rewritten before it); median of 5."""
    import torch
    import paper_2603_07169_b200 as b200sp
    A = w.A
    d_col, d_val, d_x = up(A.col_idx, dev), up(stored(A.vals, dtype), dev), up(stored(w.x, dtype), dev)
    flush = torch.empty(max(2 * l2_bytes, 256 << 20) // 4, dtype=torch.float32, device=dev)
    out = torch.zeros(torch.cuda.get_device_properties(dev).multi_processor_count * 1024, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    ts = []
    for rep in range(6):
        flush.fill_(1.0)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        b200sp.b200sp_probe_spmv_gather(A.nnz, d_col, d_val, d_x, dtype, 0, out, stream)
        b.record(stream)
        b.synchronize()
        if rep:
            ts.append(a.elapsed_time(b) * 1e-3)
    ts.sort()
    return ts[len(ts) // 2]


def run_probes(dev, l2_bytes):
    """The hardware rates that bound the kernels, each measured by a library probe kernel that does nothing else (CUDA events,
    median of 7 repetitions, a buffer larger than L2 rewritten between repetitions so that every repetition starts cold)."""
    import torch
    import paper_2603_07169_b200 as b200sp
    stream = torch.cuda.current_stream()
    sink = torch.zeros(1, dtype=torch.float32, device=dev)
    flush = torch.empty(max(2 * l2_bytes, 256 << 20) // 4, dtype=torch.float32, device=dev)
    props = torch.cuda.get_device_properties(dev)
    sms = props.multi_processor_count
    clock_hz = float(getattr(props, "clock_rate", 1965000)) * 1e3      # kHz -> Hz (maximum SM clock)

    def timed(fn, reps=7):
        fn()
        ts = []
        for _ in range(reps):
            flush.fill_(1.0)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            b.synchronize()
            ts.append(a.elapsed_time(b) * 1e-3)
        ts.sort()
        return ts[len(ts) // 2]

    out = {"device": props.name, "sms": sms, "l2_mb": round(l2_bytes / 1e6, 1), "rows": []}

    def row(name, value, unit, note=""):
        out["rows"].append({"probe": name, "value": round(value, 2), "unit": unit, "note": note})

    # streaming reads
    for nbytes, label in ((1 << 30, "1 GiB"), (134_217_728, "134 MB (the CSR arrays of the uniform workload)"), (688_000_000, "688 MB (the stencil workload)")):
        buf = torch.zeros(nbytes // 4, dtype=torch.int32, device=dev)
        t = timed(lambda: b200sp.b200sp_probe_stream(buf, buf.numel() * 4, sink, stream))
        row("streaming read, 128-bit loads, %s" % label, buf.numel() * 4 / t * 1e-9, "GB/s", "%.1f us" % (t * 1e6))
        del buf
    # random gathers
    gathers = 1 << 26
    for elems, eb, smem, label in ((16384, 4, 0, "4-byte gathers, table 64 KB (fits L1)"), (1 << 20, 4, 0, "4-byte gathers, table 4 MB (fits L2, not L1)"),
                                   (1 << 22, 4, 0, "4-byte gathers, table 16 MB"), (1 << 20, 2, 0, "2-byte gathers, table 2 MB"),
                                   (8192, 4, 1, "4-byte gathers, table 32 KB held in shared memory"),
                                   (32768, 4, 1, "4-byte gathers, table 128 KB held in shared memory")):
        table = torch.zeros(elems, dtype=torch.float32 if eb == 4 else torch.int16, device=dev)
        t = timed(lambda: b200sp.b200sp_probe_gather_ex(table, elems, gathers, eb, smem, sink, stream))
        rate = gathers / t
        row("random " + label, rate * 1e-9, "G gathers/s", "%.2f per clock per SM at %d MHz" % (rate / sms / (clock_hz), int(clock_hz // 1e6)))
        del table
    # random full-line reads (SpMM's reads of B): lines in flight per group of eight lanes, in registers or through cp.async
    reads = 1 << 25
    for lines, label in ((1 << 19, "64 MB of lines (one k-slice of B of the SpMM workload)"), (1 << 17, "16 MB of lines (L2-resident)")):
        buf = torch.zeros(lines * 32, dtype=torch.int32, device=dev)
        for inflight, to_smem, gl in ((4, 0, 8), (8, 0, 8), (16, 0, 8), (4, 1, 8), (8, 1, 8), (16, 1, 8), (4, 0, 16), (4, 0, 32), (8, 0, 32)):
            nreads = reads * 8 // gl                       # the same number of bytes for every group width
            t = timed(lambda: b200sp.b200sp_probe_lines(buf, lines, nreads, sink, inflight, to_smem, stream, gl))
            row("random %d-byte reads (%d consecutive line%s) by groups of %d lanes, %d in flight per group %s, %s"
                % (gl * 16, gl // 8, "s" if gl > 8 else "", gl, inflight, "to shared memory (cp.async)" if to_smem else "to registers", label),
                nreads * gl * 16 / t * 1e-12, "TB/s", "%.1f bytes per clock per SM" % (nreads * gl * 16 / t / sms / clock_hz))
        del buf
    # the gather phase of SpMV on the workloads' own matrices, against the shared memory carved out of the unified cache
    import gen
    for name in ("c3", "c3p", "c2"):
        w = gen.workload(name)
        A = w.A
        d_col, d_val, d_x = up(A.col_idx, dev), up(np.ascontiguousarray(A.vals, np.float32), dev), up(np.ascontiguousarray(w.x, np.float32), dev)
        outv = torch.zeros(sms * 1024, dtype=torch.float32, device=dev)
        for kb in (0, 8, 16, 32, 64, 100, 164):
            t = timed(lambda: b200sp.b200sp_probe_spmv_gather(A.nnz, d_col, d_val, d_x, "f32", kb, outv, stream))
            row("gather phase of SpMV alone on %s (FP32), %d KB of shared memory carved out per SM" % (name, kb), t * 1e6, "us",
                "%.0f G gathers/s" % (A.nnz / t * 1e-9))
        del d_col, d_val, d_x, w, A
    return out


def request_bound(rec, w, dtype, gather_rate):
    """A bound from MEASURED L1-to-L2 traffic instead of one miss per nonzero: the ncu capture of this workload counts the
    sectors the L1s asked L2 for; the CSR stream's share of them arrives four sectors to a request (128-bit coalesced loads of
    whole lines), every other sector is a request of its own, and the SMs issue requests at the probe's rate."""
    if not rec or "l2_sectors_read_by_l1" not in rec or rec.get("l1_hit_pct", 0.0) > 50.0:
        return {}       # no capture, or a kernel whose gathers mostly hit L1 (and whose CSR stream arrives by bulk copies): not request-bound
    A = w.A
    e = 4 if dtype == "f32" else 2
    stream_sectors = (A.nnz * (4 + e) + (A.m + 1) * 4) / 32.0
    sectors = float(rec["l2_sectors_read_by_l1"])
    requests = max(sectors - stream_sectors, 0.0) + stream_sectors / 4.0
    return {"request_bound_ms": round(requests / gather_rate * 1e3, 5), "l1_hit_pct_ncu": rec.get("l1_hit_pct"),
            "request_bound_note": "L1-to-L2 requests counted by ncu (%.3g sectors, CSR stream four to a request) at the probe's request rate" % sectors}


_LINES_RATE = {}


def probe_lines_rate(dev, lines=1 << 19) -> float:
    """Bytes per second of random 128-byte line reads by groups of eight lanes with four lines in flight per group (the access
    pattern of the k-sliced SpMM kernel's reads of B), from a buffer of `lines` lines; measured once per process."""
    import torch
    import paper_2603_07169_b200 as b200sp
    if dev not in _LINES_RATE:
        buf = torch.zeros(lines * 32, dtype=torch.int32, device=dev)
        sink = torch.zeros(1, dtype=torch.float32, device=dev)
        stream = torch.cuda.current_stream()
        reads = 1 << 25
        for _ in range(2):
            b200sp.b200sp_probe_lines(buf, lines, reads, sink, 4, 0, stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(3):
            b200sp.b200sp_probe_lines(buf, lines, reads, sink, 4, 0, stream)
        b.record(stream)
        b.synchronize()
        _LINES_RATE[dev] = 3 * reads * 128 / (a.elapsed_time(b) * 1e-3)
        del buf
    return _LINES_RATE[dev]


class CuSparse:
    """cuSPARSE generic API through ctypes, timed on the same device buffers as a comparison point only."""
    R_32F, R_16BF, IDX_32I, ORDER_ROW = 0, 14, 2, 2

    def __init__(self):
        import ctypes
        self.c = ctypes
        self.lib = None
        for name in ("libcusparse.so.12", "libcusparse.so"):
            try:
                self.lib = ctypes.CDLL(name)
                break
            except OSError:
                continue
        if self.lib is None:
            raise OSError("libcusparse not found")
        self.h = ctypes.c_void_p()
        self._ck(self.lib.cusparseCreate(ctypes.byref(self.h)))

    def _ck(self, rc):
        if rc != 0:
            raise RuntimeError("cuSPARSE status %d" % rc)

    def time(self, sets, w, dtype, steps, stream):
        """Mean time per call (ms) of cusparseSpMV / cusparseSpMM over the device sets `sets` in rotation (cold L2 like our own
        timing; buffer sizing and preprocess excluded)."""
        import torch
        c, L = self.c, self.lib
        A = w.A
        vt = self.R_32F if dtype == "f32" else self.R_16BF
        vp = c.c_void_p
        if not isinstance(sets, (list, tuple)):
            sets = [sets]
        self._ck(L.cusparseSetStream(self.h, vp(stream.cuda_stream)))
        alpha, beta = c.c_float(w.alpha), c.c_float(w.beta)
        runs, keep, mats = [], [], []
        for s in sets:
            mat = vp()
            self._ck(L.cusparseCreateCsr(c.byref(mat), c.c_int64(A.m), c.c_int64(A.n), c.c_int64(A.nnz), vp(s.rp.data_ptr()), vp(s.ci.data_ptr()),
                                         vp(s.va.data_ptr()), self.IDX_32I, self.IDX_32I, 0, vt))
            mats.append(mat)
            size = c.c_size_t(0)
            out = s.out.clone()
            if w.k:
                dB, dC = vp(), vp()
                self._ck(L.cusparseCreateDnMat(c.byref(dB), c.c_int64(A.n), c.c_int64(w.k), c.c_int64(w.k), vp(s.inp.data_ptr()), vt, self.ORDER_ROW))
                self._ck(L.cusparseCreateDnMat(c.byref(dC), c.c_int64(A.m), c.c_int64(w.k), c.c_int64(w.k), vp(out.data_ptr()), vt, self.ORDER_ROW))
                args = (self.h, 0, 0, c.byref(alpha), mat, dB, c.byref(beta), dC, self.R_32F, 0)
                self._ck(L.cusparseSpMM_bufferSize(*args, c.byref(size)))
                buf = torch.empty(max(size.value, 16), dtype=torch.uint8, device=s.va.device)
                if hasattr(L, "cusparseSpMM_preprocess"):
                    self._ck(L.cusparseSpMM_preprocess(*args, vp(buf.data_ptr())))
                runs.append(lambda args=args, buf=buf: L.cusparseSpMM(*args, vp(buf.data_ptr())))
            else:
                dX, dY = vp(), vp()
                self._ck(L.cusparseCreateDnVec(c.byref(dX), c.c_int64(A.n), vp(s.inp.data_ptr()), vt))
                self._ck(L.cusparseCreateDnVec(c.byref(dY), c.c_int64(A.m), vp(out.data_ptr()), vt))
                args = (self.h, 0, c.byref(alpha), mat, dX, c.byref(beta), dY, self.R_32F, 0)
                self._ck(L.cusparseSpMV_bufferSize(*args, c.byref(size)))
                buf = torch.empty(max(size.value, 16), dtype=torch.uint8, device=s.va.device)
                if hasattr(L, "cusparseSpMV_preprocess"):
                    self._ck(L.cusparseSpMV_preprocess(*args, vp(buf.data_ptr())))
                runs.append(lambda args=args, buf=buf: L.cusparseSpMV(*args, vp(buf.data_ptr())))
            keep.append((out, buf))
        for i in range(max(3, len(runs))):
            self._ck(runs[i % len(runs)]())
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(steps):
            self._ck(runs[i % len(runs)]())
        b.record(stream)
        b.synchronize()
        for mat in mats:
            L.cusparseDestroySpMat(mat)
        del keep
        return a.elapsed_time(b) / steps


def paper_sweep(quick, dev, l2_bytes):
    """The experiment the paper ran for this operator (Table 6, tasks 12 / 13; Fig. 3a): its own sizes, speed-up over a
    naive baseline kernel and the complexity-weighted score P = sum T(N_i) S_i / sum T(N_i) (Section 3.3, Eq. 1-2),
    for this library and for cuSPARSE.  T(N) = nnz for SpMV and nnz * K for SpMM, as in the table.  `quick` leaves out the
    two largest SpMM sizes (2^16 and 2^18 rows).  Returns the record."""
    import torch
    import gen
    import paper_2603_07169_b200 as b200sp
    stream = torch.cuda.current_stream()
    try:
        cusp = CuSparse()
    except Exception:
        cusp = None

    def timed(fn, sets, steps):
        for s_ in sets:          # every operand copy once: plans are built and cached here, not in the timed loop
            fn(s_)
        for i in range(3):
            fn(sets[i % len(sets)])
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(steps):
            fn(sets[i % len(sets)])
        b.record(stream)
        b.synchronize()
        return a.elapsed_time(b) / steps * 1e3   # us

    def timed_graph(fn, sets, calls=100, replays=5):
        """Per-call device time (us) of `calls` back-to-back calls replayed from a CUDA graph: no host launch cost."""
        for s_ in sets:
            fn(s_)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            cap = torch.cuda.current_stream()
            with torch.cuda.graph(g, stream=side):
                for i in range(calls):
                    fn(sets[i % len(sets)], cap)
        torch.cuda.current_stream().wait_stream(side)
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(replays):
            g.replay()
        b.record()
        b.synchronize()
        return a.elapsed_time(b) / (replays * calls) * 1e3

    out = {}
    spmm_rows = [2 ** 10, 2 ** 12, 2 ** 14, 2 ** 16, 2 ** 18]
    for op, rows_list, k in (("spmv", [2 ** e for e in range(10, 16)], 0), ("spmm", spmm_rows if not quick else spmm_rows[:3], 4096)):
        for dtype in ("f32", "bf16"):
            rec = {"rows": [], "nnz": [], "ours_us": [], "naive_us": [], "cusparse_us": []}
            for rows in rows_list:
                A = gen.paper_uniform(rows, 2048, 0.01, seed=rows + k)
                w = gen.Workload("paper", A, x=gen.uniform(2048, -1.0, 1.0, 7, 1), B=(gen.normal(2048 * k, 7, 2) if k else None), k=k)
                e = 4 if dtype == "f32" else 2
                abytes = gen.algorithmic_bytes(A.m, A.n, A.nnz, e, 0.0, k)
                R = int(max(2, min(64, -(-2 * l2_bytes // abytes), (6 << 30) // abytes)))
                sets = [DeviceSet(w, dtype, dev) for _ in range(R)]
                if k:
                    ours = lambda s, st=stream: b200sp.spmm_csr(A.m, A.n, A.nnz, k, s.rp, s.ci, s.va, s.inp, s.out, 1.0, 0.0, dtype, st)
                    naive = lambda s, st=stream: b200sp.b200sp_spmm_naive(A.m, A.n, A.nnz, k, s.rp, s.ci, s.va, s.inp, s.out, 1.0, 0.0, dtype, st)
                else:
                    ours = lambda s, st=stream: b200sp.spmv_csr(A.m, A.n, A.nnz, s.rp, s.ci, s.va, s.inp, s.out, 1.0, 0.0, dtype, st)
                    naive = lambda s, st=stream: b200sp.b200sp_spmv_naive(A.m, A.n, A.nnz, s.rp, s.ci, s.va, s.inp, s.out, 1.0, 0.0, dtype, st)
                steps = 200 if not k else max(5, min(100, int(2e11 / (A.nnz * k))))
                rec["rows"].append(rows); rec["nnz"].append(A.nnz)
                if k:
                    rec["ours_us"].append(round(timed(ours, sets, steps), 3))
                    rec["naive_us"].append(round(timed(naive, sets, max(3, steps // 4)), 3))
                else:   # a few microseconds per call: replay from a CUDA graph so that the host launch path is not what is timed
                    rec["ours_us"].append(round(timed_graph(ours, sets), 3))
                    rec["naive_us"].append(round(timed_graph(naive, sets), 3))
                    rec.setdefault("ours_host_launched_us", []).append(round(timed(ours, sets, steps), 3))
                cu = None
                if cusp is not None:
                    try:
                        cu = round(cusp.time(sets, w, dtype, steps, stream) * 1e3, 3)
                    except Exception:
                        cu = None
                rec["cusparse_us"].append(cu)
                del sets
                b200sp.b200sp_cache_clear()
                torch.cuda.empty_cache()
            T = [n * max(k, 1) for n in rec["nnz"]]
            S = [n / o for n, o in zip(rec["naive_us"], rec["ours_us"])]
            rec["speedup_ours"] = [round(v, 3) for v in S]
            rec["P_ours"] = round(sum(t * v for t, v in zip(T, S)) / sum(T), 3)
            if all(c for c in rec["cusparse_us"]):
                Sc = [n / c for n, c in zip(rec["naive_us"], rec["cusparse_us"])]
                rec["speedup_cusparse"] = [round(v, 3) for v in Sc]
                rec["P_cusparse"] = round(sum(t * v for t, v in zip(T, Sc)) / sum(T), 3)
            out["%s_%s" % (op, dtype)] = rec
    out["note"] = ("rows x 2048 at density 0.01 (K = 4096 for SpMM%s); speed-ups over the naive one-thread-per-row (per-entry) kernel; "
                   "P per the paper's Eq. 1-2 with T = nnz (x K); operands rotate over independent copies; SpMV ours / naive are per-call "
                   "device times of 100 calls replayed from a CUDA graph, cuSPARSE and SpMM are launched from the host"
                   % (", SpMM rows 2^10, 2^12, 2^14 only" if quick else ""))
    return out


def run_reference(args):
    """The oracle, as it stands, on the host cores, on the headline workload (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import gen
    import oracle
    w = gen.workload("c2")
    A = w.A
    abytes = gen.algorithmic_bytes(A.m, A.n, A.nnz, 4, w.beta)
    nt = oracle.max_threads()
    run = lambda: oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, w.x, w.y0, w.alpha, w.beta, "f32", nthreads=nt)
    t = time.perf_counter(); run(); first = time.perf_counter() - t
    steps, warmup = args.steps, args.warmup
    budget = 150.0
    if first * (steps + warmup) > budget:      # keep the whole run within a few minutes
        steps = max(1, int(budget / first) - warmup)
    for _ in range(warmup):
        run()
    t = time.perf_counter()
    for _ in range(steps):
        run()
    dt = (time.perf_counter() - t) / steps
    val = abytes / dt * 1e-9
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": "c2: CSR SpMV m=n=2^20, 16 nnz/row uniform, FP32 storage, alpha=1.5 beta=0.5",
                       "gflops": 2.0 * A.nnz / dt * 1e-9},
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": nt, "kind": "oracle",
                             "sample": "whole workload per step (16.8 M nonzeros), OpenMP over rows"},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="only the headline workload")
    ap.add_argument("--workload", default="c2", help="headline workload (default c2)")
    ap.add_argument("--dtype", default="f32")
    ap.add_argument("--paper-sweep", action="store_true", help="the paper's own SpMV / SpMM sizes with speed-up over a naive kernel and its score P")
    ap.add_argument("--quick", action="store_true", help="with --paper-sweep: skip the two largest SpMM sizes")
    ap.add_argument("--probes", action="store_true", help="measure the hardware rates behind the secondary bounds and print them")
    ap.add_argument("--opt", action="append", default=[], help="library tuning switch name=value (b200sp_set_option), repeatable")
    ap.add_argument("--profile", action="store_true",
                    help="short run for a profiler: the timed loop of one workload only (no clock loop, e2e, extras, CPU baseline)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    import gen
    import paper_2603_07169_b200 as b200sp

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    barrier = None
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
        barrier = lambda: (dist.barrier(), torch.cuda.synchronize())
    for o in args.opt:
        name, val = o.split("=")
        b200sp.b200sp_set_option(name, int(val))
    peak, peak_kind = measured_peaks()
    l2 = torch.cuda.get_device_properties(local).L2_cache_size
    steps, warmup = max(args.steps, 1), max(args.warmup, 3)

    if args.paper_sweep:
        if rank == 0:
            print(json.dumps({"paper_sweep": paper_sweep(args.quick, dev, l2)}))
        return
    if args.probes:
        if rank == 0:
            print(json.dumps({"probes": run_probes(dev, l2)}))
        return
    sampler = ClockSampler(local)
    sampler.start()
    w = gen.workload(args.workload)
    dtype = args.dtype
    try:
        cusp = CuSparse() if (rank == 0 and not args.profile) else None
    except Exception:  # pragma: no cover
        cusp = None
    head = measure(w, dtype, steps, warmup, dev, l2, barrier, cusparse=cusp)
    if args.profile:
        sampler.stop()
        print(json.dumps({"profile_run": args.workload, "dtype": dtype, "ms_per_step": head["ms_per_step"], "gbs": head["gbs"],
                          "frac": head["gbs"] / peak, "launches": head["launches"]}))
        return
    # keep the same loop running for about a second so that the clock sampler sees it under load
    t_end = time.perf_counter() + 1.0
    i = 0
    while time.perf_counter() < t_end:
        for _ in range(50):
            head["_call"](head["_sets"][i % head["copies"]]); i += 1
        torch.cuda.synchronize()
    t_load_end = time.perf_counter()
    clocks = sampler.summary(head["t0"], t_load_end)

    # max over ranks of the timed region
    ms_step, value = aggregate_over_ranks(head["ms_total"], head["algorithmic_bytes"], steps, world, dist if world > 1 else None, dev)
    gather_rate = probe_gather_rate(w.A.n, dev) if not w.k else None
    try:
        gather_alone_ms = probe_gather_phase(w, dtype, dev, l2) * 1e3 if not w.k else None
    except Exception:  # pragma: no cover
        gather_alone_ms = None

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    A = w.A
    hs = [torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
          for a in (A.row_ptr, A.col_idx, stored(A.vals, dtype), stored(w.B if w.k else w.x, dtype))]
    kk = max(w.k, 1)
    hy = (torch.from_numpy(stored(w.y0, dtype).view(np.int16) if dtype == "bf16" else stored(w.y0, dtype)).pin_memory()
          if (w.beta != 0 and w.y0 is not None) else torch.zeros(A.m * kk, dtype=torch.float32 if dtype == "f32" else torch.int16).pin_memory())
    stream = torch.cuda.current_stream()

    def host_call():
        if w.k:
            b200sp.spmm_csr_host(A.m, A.n, A.nnz, w.k, hs[0], hs[1], hs[2], hs[3], hy, w.alpha, w.beta, dtype, stream)
        else:
            b200sp.spmv_csr_host(A.m, A.n, A.nnz, hs[0], hs[1], hs[2], hs[3], hy, w.alpha, w.beta, dtype, stream)

    e2e_steps = max(3, min(steps, 10))
    for _ in range(3):
        host_call()
    torch.cuda.synchronize()
    if barrier:
        barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        host_call()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    if world > 1:
        t = torch.tensor([e2e_s], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    el = 4 if dtype == "f32" else 2
    h2d = sum(int(h.numel() * h.element_size()) for h in hs) + (A.m * kk * el if w.beta != 0 else 0)
    d2h = A.m * kk * el
    e2e = {"value": world * head["algorithmic_bytes"] / e2e_s * 1e-9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s * 1e3, "steps": e2e_steps,
           "note": "spmv_csr_host: pinned host buffers, H2D of all CSR arrays and operands, plan, kernels, D2H of y, sync"}

    # second end-to-end figure: matrix resident on the device, x and y in pinned host memory (an iterative method's step)
    if not w.k:
        res_set = DeviceSet(w, dtype, dev)
        vec_call = lambda: b200sp.spmv_csr_vec_host(A.m, A.n, A.nnz, res_set.rp, res_set.ci, res_set.va, hs[3], hy, w.alpha, w.beta, dtype, stream)
        for _ in range(3):
            vec_call()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(50):
            vec_call()
        torch.cuda.synchronize()
        vs = (time.perf_counter() - t0) / 50
        e2e["matrix_resident"] = {"value": world * head["algorithmic_bytes"] / vs * 1e-9, "unit": "GB/s", "ms_per_step": vs * 1e3,
                                  "h2d_bytes_per_step": A.n * el + (A.m * el if w.beta != 0 else 0), "d2h_bytes_per_step": A.m * el,
                                  "note": "spmv_csr_vec_host: CSR arrays stay on the device, x (and y0) copied in and y copied out every step"}
        del res_set
        b200sp.b200sp_cache_clear()

    # ---- other workloads (bounded): same protocol, fewer steps
    extras = {}
    if not args.no_extras and rank == 0:
        del head["_sets"], head["_call"]
        torch.cuda.empty_cache()
        todo = [("c2", "bf16"), ("c3", "f32"), ("c3p", "f32"), ("c4", "bf16"), ("c1", "f32"), ("c5k64", "f32"), ("c5k64", "bf16"),
                ("c5k256", "f32"), ("c5k256", "bf16")]
        cache = {args.workload: w}
        window_ab = {}
        for name, dt in todo:
            if (name, dt) == (args.workload, dtype):
                continue
            try:
                ww = cache.get(name) or gen.workload(name)
                cache = {name: ww}
                r = measure(ww, dt, min(steps, 50), 5, dev, l2, cusparse=cusp)
                extras["%s_%s" % (name, dt)] = {
                    "ms_per_step": round(r["ms_per_step"], 5), "ms_isolated_median": round(r["ms_per_step_isolated_median"], 5),
                    "ms_warm_l2": round(r["ms_per_step_warm"], 5),
                    "gbs": round(r["gbs"], 1), "frac_of_hbm": round(r["gbs"] / peak, 4), "gflops": round(r["gflops"], 1),
                    "algorithmic_bytes": r["algorithmic_bytes"], "nnz": r["nnz"], "copies": r["copies"],
                    "plan_ms_first_call": round(r["plan_ms_first_call"], 3),
                    "cusparse_ms": round(r["cusparse_ms"], 5) if isinstance(r["cusparse_ms"], float) else r["cusparse_ms"]}
                ck = sampler.summary(r["t0"], r["t1"])      # SM clock and throttle reasons sampled while THIS workload was timed
                extras["%s_%s" % (name, dt)]["clocks"] = {"sm_mhz": ck.get("sm_mhz"), "reasons": ck.get("reasons"), "samples": ck.get("samples")}
                if name == "c1":   # launch-latency regime: per-call device time from a CUDA graph, and the floors on the same box
                    extras["c1_f32"].update(latency_floor(r["_call"], r["_sets"], dev, r["algorithmic_bytes"]))
                if not ww.k:   # SpMV: time at the measured L1-miss gather rate for this x
                    rate = probe_gather_rate(ww.A.n, dev)
                    ex_ = extras["%s_%s" % (name, dt)]
                    ex_["gather_bound_ms"] = round(ww.A.nnz / rate * 1e3, 5)
                    ex_.update(request_bound(ncu_record(name, dt), ww, dt, rate))
                    if name in ("c2", "c3", "c3p"):   # the floor on the matrix itself: a loop that only gathers (no rows, no y)
                        ex_["gather_phase_alone_ms"] = round(probe_gather_phase(ww, dt, dev, l2) * 1e3, 5)
                else:          # SpMM: time of its reads of B (nnz * k * e bytes, one 128-byte line per nonzero and slice) at the measured rate of such reads
                    lr = probe_lines_rate(dev)
                    ex_ = extras["%s_%s" % (name, dt)]
                    ex_["line_read_bound_ms"] = round(ww.A.nnz * ww.k * (4 if dt == "f32" else 2) / lr * 1e3, 5)
                    ex_["line_read_rate_tbs"] = round(lr * 1e-12, 2)
                del r
                b200sp.b200sp_cache_clear()
                torch.cuda.empty_cache()
            except Exception as ex:  # pragma: no cover
                extras["%s_%s" % (name, dt)] = {"error": repr(ex)}
            if (name, dt) in (("c3", "f32"), ("c2", "bf16"), ("c5k64", "f32")) and "ms_per_step" in extras.get("%s_%s" % (name, dt), {}):
                try:   # the L2 access-policy window on the gathered operand, off / on
                    b200sp.b200sp_set_option("x_l2_window", 1)
                    r1 = measure(ww, dt, min(steps, 50), 5, dev, l2)
                    window_ab["%s_%s" % (name, dt)] = {"window_off_ms": extras["%s_%s" % (name, dt)]["ms_per_step"], "window_on_ms": round(r1["ms_per_step"], 5)}
                    del r1
                except Exception as ex:  # pragma: no cover
                    window_ab["%s_%s" % (name, dt)] = {"error": repr(ex)}
                finally:
                    b200sp.b200sp_set_option("x_l2_window", 0)
                    b200sp.b200sp_cache_clear()
                    torch.cuda.empty_cache()
        # SpMM on the power-law matrix (not one of the five configurations): the nnz-balanced kernel that the plan picks for uneven rows
        try:
            cache = {}
            wpl = gen.workload("c3k64")
            lr = probe_lines_rate(dev)
            for dt in ("f32", "bf16"):
                r = measure(wpl, dt, min(steps, 20), 3, dev, l2, cusparse=cusp)
                extras["c3k64_%s" % dt] = {
                    "ms_per_step": round(r["ms_per_step"], 5), "gbs": round(r["gbs"], 1), "frac_of_hbm": round(r["gbs"] / peak, 4),
                    "algorithmic_bytes": r["algorithmic_bytes"], "nnz": r["nnz"], "copies": r["copies"],
                    "cusparse_ms": round(r["cusparse_ms"], 5) if isinstance(r["cusparse_ms"], float) else r["cusparse_ms"],
                    "line_read_bound_ms": round(wpl.A.nnz * 64 * (4 if dt == "f32" else 2) / lr * 1e3, 5),
                    "note": "R-MAT scale 22 pattern (61 % empty rows, rows up to 57 k) times a dense 2^22 x 64 B: spmm_flat_kernel"}
                del r
                b200sp.b200sp_cache_clear()
                torch.cuda.empty_cache()
            del wpl
        except Exception as ex:  # pragma: no cover
            extras["c3k64"] = {"error": repr(ex)}
        extras["x_l2_window_ab"] = dict(window_ab, note="per-launch access-policy window (persisting hits) over x, or over B for SpMM; default off")
        # the COO and ELL front ends on the same matrices (paper tasks 8 and 14)
        for name, dt in (("c2", "f32"), ("c4", "bf16")):
            for kind in ("coo", "ell", "csc"):
                try:
                    ww = cache.get(name) or gen.workload(name)
                    cache = {name: ww}
                    r = measure_format(kind, ww, dt, min(steps, 50), dev, l2)
                    r["frac_of_hbm"] = round(r["gbs"] / peak, 4)
                    extras["%s_%s_%s" % (kind, name, dt)] = r
                    torch.cuda.empty_cache()
                except Exception as ex:  # pragma: no cover
                    extras["%s_%s_%s" % (kind, name, dt)] = {"error": repr(ex)}
        # the paper's own experiment at its sizes (Table 6, tasks 12 / 13; score P of Section 3.3), short form
        try:
            cache = {}
            sw = paper_sweep(True, dev, l2)
            extras["paper_sweep_quick"] = {k: ({kk: v[kk] for kk in ("rows", "ours_us", "naive_us", "cusparse_us", "P_ours", "P_cusparse") if kk in v}
                                               if isinstance(v, dict) else v) for k, v in sw.items()}
        except Exception as ex:  # pragma: no cover
            extras["paper_sweep_quick"] = {"error": repr(ex)}
    sampler.stop()

    # ---- CPU baseline: the oracle on the host cores, same workload (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1:
        import oracle
        nt = oracle.max_threads()
        vals_s, in_s = stored(A.vals, dtype), stored(w.B if w.k else w.x, dtype)
        y0_s = stored(w.y0, dtype) if w.beta != 0 else None
        best, best1, y_ref, S_ref = 1e30, 1e30, None, None
        if w.k:
            rows = np.arange(0, A.m, max(1, A.m // 4096), dtype=np.int64)
            run = lambda n_t: oracle.spmm_csr(A.m, A.n, w.k, A.row_ptr, A.col_idx, vals_s, in_s, y0_s, w.alpha, w.beta, dtype, rows=rows, nthreads=n_t)
            frac_rows, sample = len(rows) / A.m, "%d sampled rows of the workload" % len(rows)
        else:
            run = lambda n_t: oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, vals_s, in_s, y0_s, w.alpha, w.beta, dtype, nthreads=n_t)
            frac_rows, sample = 1.0, "whole workload, best of 3, OpenMP over rows"
        for _ in range(3):
            t = time.perf_counter(); y_ref, S_ref = run(nt); best = min(best, time.perf_counter() - t)
        t = time.perf_counter(); run(1); best1 = time.perf_counter() - t
        cpu = {"value": head["algorithmic_bytes"] * frac_rows / best * 1e-9, "unit": "GB/s", "cores": nt, "kind": "oracle",
               "sample": sample, "ms": best * 1e3, "ms_single_thread": best1 * 1e3}

    if rank == 0:
        config = {"workload": "%s: %s" % (args.workload, {
            "c2": "CSR SpMV m=n=2^20, exactly 16 nnz/row uniform sorted columns, vals N(0,1), alpha=1.5 beta=0.5"}.get(args.workload, w.A.name)),
            "m": A.m, "n": A.n, "nnz": A.nnz, "k": w.k, "alpha": w.alpha, "beta": w.beta,
            "algorithmic_bytes_per_step": head["algorithmic_bytes"], "gflops": world * head["gflops"],
            "l2": "steps rotate over %d device copies of all operands (%.0f MB in total, L2 is %.0f MB); no flush in the timed region"
                  % (head["copies"], head["copies"] * head["algorithmic_bytes"] / 1e6, l2 / 1e6),
            "plan": "cached per row_ptr; first call incl. plan %.3f ms (excluded)" % head["plan_ms_first_call"],
            "ms_per_step_isolated_median": head["ms_per_step_isolated_median"],
            "ms_per_step_warm_l2": head["ms_per_step_warm"],
            "parallelism": "replicas only (single-GPU path)" if world > 1 else "1 GPU"}
        achieved = head["algorithmic_bytes"] / (head["ms_total"] / steps) * 1e-6
        line = {"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": warmup,
                "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dtype,
                "data": "synthetic", "config": config, "clocks": clocks, "e2e": e2e,
                "gpu_launches": int(head["launches"]),
                "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                             "traffic": ncu_traffic(args.workload, dtype), "peak_kind": "of " + peak_kind,
                             "frac_of_nominal_7700": achieved / 7700.0,
                             "note": "algorithmic bytes per step over event time per step (the step is the SpMV kernel; plan cached)",
                             "binding_bound": "secondary" if (gather_rate is not None and A.nnz / gather_rate * 1e3 > head["algorithmic_bytes"] / peak * 1e-6) else "hbm",
                             "secondary": None if gather_rate is None else {
                                 "bound": "L1-miss gather (one L2 request per random x read)", "gathers_per_s": gather_rate,
                                 "ms_at_bound": A.nnz / gather_rate * 1e3, "frac_of_bound": (A.nnz / gather_rate * 1e3) / (head["ms_total"] / steps),
                                 "note": "measured live with b200sp_probe_gather on a table the size of x",
                                 "gather_phase_alone_ms": gather_alone_ms,
                                 "gather_phase_note": "b200sp_probe_spmv_gather on this workload's own col_idx / vals / x, started cold: a loop that only gathers (no row sums, no y)"}},
                "cusparse": {"ms_per_step": head["cusparse_ms"], "note": "cusparseSpMV/SpMM, default algorithm, preprocess excluded, over the same rotated operand copies (cold L2); comparison point only"},
                "cpu_baseline": cpu, "extra": extras}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
