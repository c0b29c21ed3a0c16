"""Three-way bottleneck classification of a profiled kernel, after the paper's hardware analysis filter
(Section 4.2, Table 2; thresholds from Appendix A, "Bottleneck Classification Logic"):

    compute bound            Compute (SM) Throughput > 30 %
    memory latency bound     Compute < 30 %, DRAM Throughput < 30 % and Memory Throughput < 30 %
    memory bandwidth bound   Compute < 30 % and (DRAM Throughput > 30 % or Memory Throughput > 30 %)

and the four metrics the table keeps for each class.  Input is Nsight Compute's raw page exported as CSV
(``ncu -i report.ncu-rep --page raw --csv``); this module only post-processes text, it launches nothing.

    python -m paper_2603_07169_b200.bottleneck raw.csv
"""
from __future__ import annotations

import csv
import sys
from typing import Dict, Iterable, List, Optional

THRESHOLD = 30.0   # percent; the paper's Otsu-calibrated cut for all three throughputs

# Nsight Compute metric names behind the paper's section labels
COMPUTE_TH = "sm__throughput.avg.pct_of_peak_sustained_elapsed"                      # Compute (SM) Throughput
DRAM_TH = "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed"                   # DRAM Throughput
MEMORY_TH = "gpu__compute_memory_throughput.avg.pct_of_peak_sustained_elapsed"       # Memory Throughput

FILTERED = {
    "compute": ["sm__throughput.avg.pct_of_peak_sustained_elapsed",                  # Compute (SM) Throughput
                "smsp__issue_active.avg.pct_of_peak_sustained_active",               # Issue Slots Busy
                "sm__inst_executed.avg.per_cycle_active",                            # Executed Ipc Active
                "sm__instruction_throughput.avg.pct_of_peak_sustained_active"],      # SM Busy
    "latency": ["lts__t_sector_hit_rate.pct",                                        # L2 Hit Rate
                "l1tex__t_sector_hit_rate.pct",                                      # L1/TEX Hit Rate
                "sm__inst_executed.avg.per_cycle_elapsed",                           # Executed Ipc Elapsed
                "gpu__compute_memory_access_throughput.avg.pct_of_peak_sustained_elapsed"],  # Mem Busy
    "bandwidth": ["gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",          # DRAM Throughput
                  "gpu__compute_memory_throughput.avg.pct_of_peak_sustained_elapsed",  # Memory Throughput
                  "gpu__compute_memory_request_throughput.avg.pct_of_peak_sustained_elapsed",  # Max Bandwidth
                  "sm__memory_throughput.avg.pct_of_peak_sustained_elapsed"],        # Mem Pipes Busy
}


def classify(compute_th: float, dram_th: float, memory_th: float, threshold: float = THRESHOLD) -> str:
    """'compute', 'latency' or 'bandwidth' from the three throughputs in percent of peak."""
    if compute_th > threshold:
        return "compute"
    if dram_th < threshold and memory_th < threshold:
        return "latency"
    return "bandwidth"


def _num(text: str) -> Optional[float]:
    try:
        return float(text.replace(",", ""))
    except (ValueError, AttributeError):
        return None


def classify_rows(rows: Iterable[List[str]]) -> List[Dict]:
    """Rows of the raw CSV page (header, units, then one row per profiled launch) -> one record per launch."""
    rows = [r for r in rows if r]
    header = rows[0]
    data = [r for r in rows[1:] if r and r[0].strip().isdigit()]
    idx = {name: i for i, name in enumerate(header)}
    out = []
    for r in data:
        get = lambda name: _num(r[idx[name]]) if name in idx and idx[name] < len(r) else None
        c, d, m = get(COMPUTE_TH), get(DRAM_TH), get(MEMORY_TH)
        rec = {"kernel": r[idx["Kernel Name"]] if "Kernel Name" in idx else "?", "compute_th": c, "dram_th": d, "memory_th": m}
        if None in (c, d, m):
            rec["class"] = None
        else:
            rec["class"] = classify(c, d, m)
            rec["filtered"] = {name: get(name) for name in FILTERED[rec["class"]]}
        out.append(rec)
    return out


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    if len(argv) != 1:
        print(__doc__)
        return 2
    with open(argv[0], newline="") as f:
        for rec in classify_rows(csv.reader(f)):
            print("%-60s compute %5s  dram %5s  memory %5s  ->  %s" % (rec["kernel"][:60], rec["compute_th"], rec["dram_th"], rec["memory_th"], rec["class"]))
            for name, v in (rec.get("filtered") or {}).items():
                print("    %-80s %s" % (name, v))
    return 0


if __name__ == "__main__":
    sys.exit(main())
