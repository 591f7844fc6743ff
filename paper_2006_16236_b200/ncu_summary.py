"""Summaries of Nsight Compute captures of the library's kernels.

    ncu -i capture.ncu-rep --page raw --csv > capture.csv
    python -m paper_2006_16236_b200.ncu_summary capture.csv --workload NAME [--traffic profiles/traffic.json]

prints one markdown table (a column per captured launch, a row per metric of interest: duration, DRAM bytes
and throughput, tensor-pipe and XU-pipe activity, issue rate, instruction-cache hit rate, registers) and,
with --traffic, records DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of every
kernel under the workload's name in the JSON file that bench.py reads its `roofline.traffic` from.
`--long` reads the other CSV layout ncu writes with --metrics ... --csv --log-file (one row per metric).
"""
from __future__ import annotations

import argparse
import csv
import json
import os
import re
import subprocess
import sys

ROWS = [
    ("gpu__time_duration.sum", "duration under ncu"),
    ("launch__registers_per_thread", "registers / thread"),
    ("launch__block_size", "block size"),
    ("launch__grid_size", "grid size"),
    ("dram__bytes_read.sum", "DRAM read"),
    ("dram__bytes_write.sum", "DRAM write"),
    ("gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "DRAM throughput, % of peak"),
    ("lts__t_bytes.sum", "L2 traffic"),
    ("sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed", "tensor pipe active, % of elapsed cycles"),
    ("sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active", "tensor pipe active, % of active cycles"),
    ("sm__inst_executed_pipe_tensor_subpipe_hmma.avg.pct_of_peak_sustained_active", "tensor (hmma) instructions, % of peak issue"),
    ("sm__inst_executed_pipe_xu.avg.pct_of_peak_sustained_elapsed", "XU pipe (ex2), % of peak"),
    ("smsp__issue_active.avg.per_cycle_active", "issue slots used per cycle"),
    ("smsp__inst_executed.sum", "warp instructions"),
    ("sm__icc_request_hit_rate.pct", "SM instruction cache hit rate, %"),
    ("sm__warps_active.avg.pct_of_peak_sustained_active", "warps active, % of peak"),
]


def short_name(kernel: str) -> str:
    m = re.search(r"([A-Za-z_0-9]+_kernel)", kernel)
    return m.group(1) if m else kernel[:40]


def read_wide(path):
    """`--page raw --csv`: a header row, a units row, one row per launch."""
    rows = list(csv.reader(open(path)))
    rows = [r for r in rows if len(r) > 10]
    hdr, units, data = rows[0], rows[1], rows[2:]
    col = {h: i for i, h in enumerate(hdr)}
    out = []
    for r in data:
        d = {"kernel": short_name(r[col["Kernel Name"]])}
        for key, _ in ROWS:
            if key in col:
                d[key] = (r[col[key]], units[col[key]])
        out.append(d)
    return out


def read_long(path):
    """`--metrics ... --csv --log-file`: one row per (launch, metric)."""
    launches = {}
    for r in csv.DictReader(line for line in open(path) if line.startswith('"')):
        d = launches.setdefault(r["ID"], {"kernel": short_name(r["Kernel Name"]), "launch__grid_size": (r["Grid Size"], "")})
        d[r["Metric Name"]] = (r["Metric Value"], r["Metric Unit"])
    return [launches[k] for k in sorted(launches, key=int)]


def to_bytes(value, unit):
    scale = {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}.get(unit)
    return None if scale is None else float(value.replace(",", "")) * scale


def fmt(value, unit):
    try:
        x = float(value.replace(",", ""))
    except ValueError:
        return value
    if unit in ("byte", "Kbyte", "Mbyte", "Gbyte"):
        return f"{to_bytes(value, unit) / 1e6:.1f} MB"
    if unit in ("ns", "us", "ms", "second"):
        us = x * {"ns": 1e-3, "us": 1.0, "ms": 1e3, "second": 1e6}[unit]
        return f"{us:.1f} us"
    if abs(x) >= 1e6:
        return f"{x / 1e6:.1f} M"
    return f"{x:.2f}".rstrip("0").rstrip(".") + ({"%": " %"}.get(unit, ""))


def git_head():
    try:
        root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
        return subprocess.run(["git", "rev-parse", "--short", "HEAD"], cwd=root, capture_output=True, text=True).stdout.strip()
    except OSError:
        return ""


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("csv")
    ap.add_argument("--workload", required=True)
    ap.add_argument("--long", action="store_true")
    ap.add_argument("--traffic", help="JSON file to record DRAM bytes per launch in")
    ap.add_argument("--pick", help="only launches whose grid size equals this (e.g. one batch size of the decode kernel)")
    args = ap.parse_args()
    launches = read_long(args.csv) if args.long else read_wide(args.csv)
    if args.pick:
        launches = [d for d in launches if d.get("launch__grid_size", ("", ""))[0].strip("() ").split(",")[0] == args.pick]
    if not launches:
        sys.exit("no launches in " + args.csv)
    if args.long and len(launches) > 6:         # many launches of one kernel: average them
        keys = [k for k, _ in ROWS if all(k in d for d in launches)]
        mean = {"kernel": launches[0]["kernel"] + f" (mean of {len(launches)} launches)"}
        for k in keys:
            try:
                mean[k] = (str(sum(float(d[k][0].replace(",", "")) for d in launches) / len(launches)), launches[0][k][1])
            except ValueError:
                mean[k] = launches[0][k]
        launches = [mean]
    print("| metric | " + " | ".join(d["kernel"] for d in launches) + " |")
    print("|---|" + "---|" * len(launches))
    for key, label in ROWS:
        if any(key in d for d in launches):
            print(f"| {label} (`{key}`) | " + " | ".join(fmt(*d[key]) if key in d else "" for d in launches) + " |")
    tr = ["" if "dram__bytes_read.sum" not in d else
          f"{(to_bytes(*d['dram__bytes_read.sum']) + to_bytes(*d['dram__bytes_write.sum'])) / 1e6:.1f} MB" for d in launches]
    print("| traffic = read + write | " + " | ".join(tr) + " |")
    if args.traffic:
        try:
            doc = json.load(open(args.traffic))
        except (OSError, ValueError):
            doc = {}
        doc["source"] = "ncu dram__bytes_read.sum + dram__bytes_write.sum, one launch per kernel, summarised under profiles/"
        doc.setdefault("commit", {})[args.workload] = git_head()
        per = doc.setdefault("bytes_per_launch", {}).setdefault(args.workload, {})
        for d in launches:
            if "dram__bytes_read.sum" in d:
                name = d["kernel"].split(" ")[0]
                per[name] = int(to_bytes(*d["dram__bytes_read.sum"]) + to_bytes(*d["dram__bytes_write.sum"]))
        with open(args.traffic, "w") as f:
            json.dump(doc, f, indent=1, sort_keys=True)
            f.write("\n")


if __name__ == "__main__":
    main()
