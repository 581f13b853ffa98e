"""Turns the raw CSV page of an ncu capture into the tracked summary bench.py reads.

    ncu -i capture.ncu-rep --page raw --csv > raw.csv
    python -m paper_2410_20305_b200.ncu_summary raw.csv --kernel psa_bwd_kernel --workload multi-turn \
        --command "<the full ncu command that made the capture>"

Writes (or updates) profiles/ncu_traffic.json: per kernel and workload the DRAM bytes (read +
write) of one launch, averaged over the captured launches, with the digest of the kernel sources
the capture was taken from (bench.py reports the figure as null when the sources have changed
since) and the command.  Also prints the other counters of interest as a markdown table for
the profiles/*.md summary.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
OUT = os.path.join(ROOT, "profiles", "ncu_traffic.json")
TRAFFIC_SOURCES = ("psa_bwd.cu", "psa_device.cuh", "psa_plan.cpp")
SCALE = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12}
SHOW = ("gpu__time_duration.sum", "sm__cycles_elapsed.avg.per_second", "launch__grid_size", "launch__registers_per_thread",
        "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
        "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed",
        "sm__inst_executed_pipe_xu.avg.pct_of_peak_sustained_active", "sm__throughput.avg.pct_of_peak_sustained_elapsed",
        "l1tex__throughput.avg.pct_of_peak_sustained_elapsed", "lts__throughput.avg.pct_of_peak_sustained_elapsed",
        "sm__warps_active.avg.pct_of_peak_sustained_active", "dram__bytes_read.sum", "dram__bytes_write.sum",
        "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "dram__throughput.avg.pct_of_peak_sustained_elapsed",
        "smsp__inst_executed.sum")


def source_digest():
    h = hashlib.sha256()
    for name in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, "paper_2410_20305_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("raw_csv")
    ap.add_argument("--kernel", required=True, help="substring of the kernel name")
    ap.add_argument("--workload", required=True)
    ap.add_argument("--command", default="")
    ap.add_argument("--no-write", action="store_true")
    args = ap.parse_args()
    rows = [r for r in csv.reader(open(args.raw_csv)) if r]
    head = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    names, units = rows[head], rows[head + 1]
    col = {n: i for i, n in enumerate(names)}
    data = [r for r in rows[head + 2:] if len(r) == len(names) and args.kernel in r[col["Kernel Name"]]]
    if not data:
        raise SystemExit("no launch of a kernel named *%s* in %s" % (args.kernel, args.raw_csv))

    def value(r, metric):
        x = float(r[col[metric]].replace(",", ""))
        return x * SCALE.get(units[col[metric]], 1.0)

    traffic = [value(r, "dram__bytes_read.sum") + value(r, "dram__bytes_write.sum") for r in data]
    print("| counter | value (mean of %d launch(es)) | unit |\n|---|---|---|" % len(data))
    for m in SHOW:
        if m in col:
            vals = [float(r[col[m]].replace(",", "")) for r in data]
            print("| %s | %.6g | %s |" % (m, sum(vals) / len(vals), units[col[m]]))
    print("| dram bytes read + write per launch | %.1f | MB |" % (sum(traffic) / len(traffic) / 1e6))
    if args.no_write:
        return
    doc = json.load(open(OUT)) if os.path.exists(OUT) else {}
    doc.setdefault(args.kernel, {})[args.workload] = {
        "dram_bytes": sum(traffic) / len(traffic), "launches": len(data), "source_digest": source_digest(),
        "command": args.command}
    with open(OUT, "w") as f:
        json.dump(doc, f, indent=1, sort_keys=True)
        f.write("\n")


if __name__ == "__main__":
    main()
