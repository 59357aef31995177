"""Records the DRAM traffic that ncu counted for one kernel in profiles/traffic.json.

Usage (on a machine without a GPU, from an ncu report brought back from the GPU machine):

    ncu -i report.ncu-rep --page raw --csv > raw.csv
    python -m paper_2412_00061_b200.ncu_traffic raw.csv --workload c2 --kernel gemv_stream_kernel \
        --sources paper_2412_00061_b200/csrc/gemv_stream.cu paper_2412_00061_b200/csrc/gemv_stream.cuh \
        --command "<the ncu command that produced the report>"

The record holds dram__bytes_read.sum + dram__bytes_write.sum averaged over the captured
launches of the kernel, the command, and the SHA-256 of the kernel's source files: the
benchmark reports the traffic only while those files are unchanged.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def read_traffic(csv_path: str, kernel: str):
    """(mean bytes per launch, launches) over the rows of the raw page whose kernel name contains `kernel`."""
    with open(csv_path, newline="") as f:
        rows = list(csv.reader(f))
    header = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    names, units = rows[header], rows[header + 1]
    col = {n: i for i, n in enumerate(names)}
    rd, wr, kn = col["dram__bytes_read.sum"], col["dram__bytes_write.sum"], col["Kernel Name"]
    vals = []
    for r in rows[header + 2:]:
        if len(r) <= max(rd, wr) or kernel not in r[kn]:
            continue
        num = lambda i: float(r[i].replace(",", "")) * UNIT.get(units[i], 1.0)
        vals.append(num(rd) + num(wr))
    if not vals:
        raise SystemExit("no launch of %s in %s" % (kernel, csv_path))
    return sum(vals) / len(vals), len(vals)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("raw_csv")
    ap.add_argument("--workload", required=True)
    ap.add_argument("--kernel", required=True)
    ap.add_argument("--sources", nargs="+", required=True, help="source files of the kernel, relative to the repository root")
    ap.add_argument("--command", required=True)
    ap.add_argument("--out", default=os.path.join(ROOT, "profiles", "traffic.json"))
    a = ap.parse_args()
    traffic, launches = read_traffic(a.raw_csv, a.kernel)
    sha = {}
    for rel in a.sources:
        with open(os.path.join(ROOT, rel), "rb") as f:
            sha[rel] = hashlib.sha256(f.read()).hexdigest()
    try:
        with open(a.out) as f:
            data = json.load(f)
    except (OSError, ValueError):
        data = {}
    data.setdefault(a.workload, {})[a.kernel] = {
        "traffic_bytes": traffic, "launches_captured": launches, "command": a.command, "source_sha256": sha}
    with open(a.out, "w") as f:
        json.dump(data, f, indent=1, sort_keys=True)
        f.write("\n")
    print("%s / %s: %.1f MB per launch over %d launches" % (a.workload, a.kernel, traffic / 1e6, launches))


if __name__ == "__main__":
    main()
