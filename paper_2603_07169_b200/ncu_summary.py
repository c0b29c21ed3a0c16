"""Turns Nsight Compute's raw CSV page into the figures the benchmark and the summaries under profiles/ quote.

    ncu -i capture.ncu-rep --page raw --csv > capture.csv
    python -m paper_2603_07169_b200.ncu_summary capture.csv --key c3_f32 [--json profiles/traffic.json] [--md]

Per captured launch it reads the kernel name, its duration, DRAM bytes read and written, the L2 and L1 hit rates, the
sectors the L1s requested from L2 and how busy the L1-to-L2 request path was (the counter that tells a gather-bound
kernel from an HBM-bound one on this part).  With --json it stores the record of the LONGEST captured launch (the
dominant kernel) under --key in that file, which bench.py reads for `roofline.traffic`; with --md it prints a table.
The paper's bottleneck rule (its Table 2) is applied by the sibling module `bottleneck`.
"""
from __future__ import annotations

import argparse
import csv
import json
import os
import sys

FIELDS = {
    "time_us": ("gpu__time_duration.sum", 1e-3),                       # ncu reports ns
    "dram_read_bytes": ("dram__bytes_read.sum", None),
    "dram_write_bytes": ("dram__bytes_write.sum", None),
    "l2_hit_pct": ("lts__t_sector_hit_rate.pct", 1.0),
    "l1_hit_pct": ("l1tex__t_sector_hit_rate.pct", 1.0),
    "l2_sectors_read_by_l1": ("lts__t_sectors_srcunit_tex_op_read.sum", 1.0),
    "l1_to_l2_request_path_busy_pct": ("l1tex__m_l1tex2xbar_req_cycles_active.avg.pct_of_peak_sustained_elapsed", 1.0),
    "dram_throughput_pct": ("gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", 1.0),
    "registers_per_thread": ("launch__registers_per_thread", 1.0),
    "achieved_occupancy_pct": ("sm__warps_active.avg.pct_of_peak_sustained_active", 1.0),
}
UNIT_SCALE = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12,
              "ns": 1.0, "us": 1e3, "ms": 1e6, "s": 1e9, "nsecond": 1.0, "usecond": 1e3, "msecond": 1e6, "second": 1e9}


def _num(text: str) -> float:
    return float(text.replace(",", "")) if text not in ("", "n/a") else float("nan")


def read_launches(path: str):
    """One dict per captured launch.  The raw page has a header row, a row of units, then one row per launch."""
    with open(path, newline="") as f:
        rows = [r for r in csv.reader(f) if r]
    start = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    head, units = rows[start], rows[start + 1]
    col = {name: i for i, name in enumerate(head)}
    out = []
    for r in rows[start + 2:]:
        if len(r) != len(head):
            continue
        rec = {"kernel": r[col["Kernel Name"]]}
        for key, (metric, scale) in FIELDS.items():
            if metric not in col:
                continue
            v = _num(r[col[metric]])
            u = units[col[metric]]
            if key == "time_us":
                v = v * UNIT_SCALE.get(u, 1.0) * 1e-3            # to microseconds
            elif scale is None:
                v = v * UNIT_SCALE.get(u, 1.0)                   # to bytes
            rec[key] = v
        if "dram_read_bytes" in rec and "dram_write_bytes" in rec:
            rec["dram_bytes"] = rec["dram_read_bytes"] + rec["dram_write_bytes"]
        out.append(rec)
    return out


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("csv")
    ap.add_argument("--key", help="record name, e.g. c3_f32")
    ap.add_argument("--json", help="file to update with the dominant launch's record")
    ap.add_argument("--command", default="", help="the ncu command line, stored with the record")
    ap.add_argument("--md", action="store_true")
    a = ap.parse_args(argv)
    launches = read_launches(a.csv)
    if not launches:
        sys.exit("no launches in %s" % a.csv)
    top = max(launches, key=lambda r: r.get("time_us", 0.0))
    if a.md:
        print("| kernel | time us | DRAM MB | L2 hit % | L1 hit % | L2 sectors read by L1 | request path busy % |")
        print("|---|---|---|---|---|---|---|")
        for r in launches:
            print("| `%s` | %.1f | %.1f | %.1f | %.1f | %.4g | %.1f |" % (
                r["kernel"][:60], r.get("time_us", float("nan")), r.get("dram_bytes", float("nan")) / 1e6, r.get("l2_hit_pct", float("nan")),
                r.get("l1_hit_pct", float("nan")), r.get("l2_sectors_read_by_l1", float("nan")), r.get("l1_to_l2_request_path_busy_pct", float("nan"))))
    if a.json:
        if not a.key:
            sys.exit("--json needs --key")
        data = {}
        if os.path.exists(a.json):
            with open(a.json) as f:
                data = json.load(f)
        rec = {k: (int(v) if k.endswith("bytes") or k == "l2_sectors_read_by_l1" else round(v, 3)) if isinstance(v, float) else v for k, v in top.items()}
        rec["launches_captured"] = len(launches)
        if a.command:
            rec["command"] = a.command
        data[a.key] = rec
        with open(a.json, "w") as f:
            json.dump(data, f, indent=1, sort_keys=True)
            f.write("\n")
    if not a.md:
        print(json.dumps(top))


if __name__ == "__main__":
    main()
