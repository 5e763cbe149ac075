"""Turns Nsight Compute CSV output into the short text summaries kept under profiles/.

Two inputs are understood:
  * the launch list written by
        ncu --metrics gpu__time_duration.sum --clock-control none --csv --log-file launches.csv <command>
    (one row per launch and metric): prints launches, total time and share per kernel;
  * the raw page of a report,
        ncu -i report.ncu-rep --page raw --csv > raw.csv
    (one row per launch, one column per metric): prints the chosen counters per launch and, with
    --traffic NAME, rewrites the line NAME of profiles/dram_traffic.txt with the DRAM bytes (read + write)
    per call (mean per launch of each captured kernel, summed over the kernels), the figure bench.py
    reports as roofline.traffic.

    python -m paper_2209_05433_b200.ncu_summary launches.csv
    python -m paper_2209_05433_b200.ncu_summary raw.csv --kernel k_gemm_fp8 --traffic k_gemm_fp8.fprop.hidden12288
"""
from __future__ import annotations

import argparse
import csv
import os
import re
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.txt")

COUNTERS = [
    "gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum", "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "lts__t_sector_hit_rate.pct", "sm__cycles_elapsed.avg.per_second", "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed",
    "sm__throughput.avg.pct_of_peak_sustained_elapsed", "sm__warps_active.avg.pct_of_peak_sustained_active",
    "smsp__issue_active.avg.pct_of_peak_sustained_active", "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_lg_throttle_per_issue_active.ratio", "launch__registers_per_thread", "launch__grid_size", "launch__block_size",
]
SCALE = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12,
         "nsecond": 1e-9, "usecond": 1e-6, "msecond": 1e-3, "second": 1.0, "ns": 1e-9, "us": 1e-6, "ms": 1e-3, "s": 1.0}


def _number(text: str) -> float:
    return float(text.replace(",", "")) if text not in ("", "n/a") else float("nan")


def _short(name: str) -> str:
    name = re.sub(r"^void\s+", "", name)
    name = re.sub(r"\(.*$", "", name)
    return name.replace("fp8b200::gemm::", "").replace("fp8b200::", "")


def _rows(path: str):
    with open(path, newline="") as f:
        lines = [l for l in f if l.startswith('"')]              # ncu prints ==PROF== lines around the table
    return list(csv.reader(lines))


def launch_list(rows) -> str:
    head = rows[0]
    k_name, k_metric, k_unit, k_val = head.index("Kernel Name"), head.index("Metric Name"), head.index("Metric Unit"), head.index("Metric Value")
    per = {}
    for r in rows[1:]:
        if r[k_metric] != "gpu__time_duration.sum":
            continue
        t = _number(r[k_val]) * SCALE.get(r[k_unit], 1.0) * 1e6        # microseconds
        e = per.setdefault(_short(r[k_name]), [0, 0.0])
        e[0] += 1
        e[1] += t
    total = sum(v[1] for v in per.values()) or 1.0
    out = ["launches  total_us  share  kernel"]
    for name, (n, t) in sorted(per.items(), key=lambda kv: -kv[1][1]):
        out.append("%6d  %9.1f  %5.2f%%  %s" % (n, t, 100.0 * t / total, name))
    return "\n".join(out)


def raw_page(rows, kernel: str | None, traffic_key: str | None) -> str:
    head, units = rows[0], rows[1]
    k_name = head.index("Kernel Name")
    cols = [(c, head.index(c)) for c in COUNTERS if c in head]
    out, traffic, names = [], [], []
    for r in rows[2:]:
        if kernel and kernel not in r[k_name]:
            continue
        out.append("--- " + _short(r[k_name]))
        vals = {}
        for c, i in cols:
            vals[c] = (_number(r[i]), units[i])
            out.append("  %-82s %14s %s" % (c, r[i], units[i]))
        if "dram__bytes_read.sum" in vals and "dram__bytes_write.sum" in vals:
            rd = vals["dram__bytes_read.sum"][0] * SCALE.get(vals["dram__bytes_read.sum"][1], 1.0)
            wr = vals["dram__bytes_write.sum"][0] * SCALE.get(vals["dram__bytes_write.sum"][1], 1.0)
            traffic.append(rd + wr)
            names.append(_short(r[k_name]))
            out.append("  %-82s %14.4e byte" % ("dram bytes read + written", rd + wr))
    if traffic_key and traffic:
        # bytes per CALL: the mean over the launches of each kernel, summed over the kernels captured
        per_kernel = {}
        for name, t in zip(names, traffic):
            per_kernel.setdefault(name, []).append(t)
        mean = sum(sum(v) / len(v) for v in per_kernel.values())
        lines = []
        if os.path.exists(TRAFFIC_FILE):
            with open(TRAFFIC_FILE) as f:
                lines = [l.rstrip("\n") for l in f if l.split()[:1] != [traffic_key]]
        lines.append("%s %.6e   # %d captured launches of %s" % (traffic_key, mean, len(traffic), " + ".join(sorted(per_kernel))))
        with open(TRAFFIC_FILE, "w") as f:
            f.write("\n".join(lines) + "\n")
        out.append("wrote %s = %.6e to %s" % (traffic_key, mean, os.path.relpath(TRAFFIC_FILE, ROOT)))
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("csv_file")
    ap.add_argument("--kernel", default=None, help="only launches whose kernel name contains this text")
    ap.add_argument("--traffic", default=None, help="name of the line of profiles/dram_traffic.txt to rewrite")
    args = ap.parse_args()
    rows = _rows(args.csv_file)
    if not rows:
        sys.exit("no CSV rows found in " + args.csv_file)
    print(launch_list(rows) if "Metric Name" in rows[0] else raw_page(rows, args.kernel, args.traffic))


if __name__ == "__main__":
    main()
