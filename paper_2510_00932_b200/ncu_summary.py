"""Turns an ncu launch list with DRAM counters into the per-kernel traffic summary bench.py reads.

    ncu --cache-control none --clock-control none --csv --log-file opmajor_dram.csv \
        --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum \
        -k regex:"ew_vec_kernel|dot_pass1" -c 200 \
        python bench.py --steps 3 --warmup 3 --cpu-seconds 0 --e2e-steps 0 --no-shmem --no-parity --extra ""
    python -m paper_2510_00932_b200.ncu_summary opmajor_dram.csv --workload c2 \
        --command "<the ncu command above>"

bench.py's op-major region launches each kernel several times in a row; in the launch list that is a
run of consecutive launches of one kernel. For every such run (the last one per kernel) the summary
keeps the median of its launches except the first: DRAM bytes read and written and the duration.
The tuning in force (read from the library's defaults) is stored beside them, so that bench.py can
tell a capture of an older kernel from a current one. Needs no GPU.
"""
from __future__ import annotations

import argparse
import csv
import json
import re
import statistics
import sys

OP_OF_CODE = {0: "copy", 1: "scale", 2: "add", 3: "triad"}


def op_of_kernel(name: str):
    if "dot_pass1_kernel" in name or "dot_roll_kernel" in name or "dot_comp_kernel" in name:
        return "dot"
    m = re.search(r"ew_vec_kernel<[^,]+,\s*(?:\(int\))?(\d)", name)
    return OP_OF_CODE.get(int(m.group(1))) if m else None


def parse(path: str):
    """[(kernel name, {metric: value})] in launch order from ncu's --csv log."""
    rows = [r for r in csv.reader(open(path)) if len(r) > 10]
    hdr = rows[0]
    i_id, i_k, i_m, i_v = (hdr.index(c) for c in ("ID", "Kernel Name", "Metric Name", "Metric Value"))
    i_u = hdr.index("Metric Unit")
    scale = {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "ns": 1e-3, "us": 1.0, "usecond": 1.0, "ms": 1e3,
             "nsecond": 1e-3, "msecond": 1e3}
    launches: dict = {}
    for r in rows[1:]:
        d = launches.setdefault(int(r[i_id]), {"kernel": r[i_k]})
        d[r[i_m]] = float(r[i_v].replace(",", "")) * scale.get(r[i_u], 1)
    return [launches[k] for k in sorted(launches)]


def op_major_runs(launches, min_len: int = 4):
    """{op: [launch, ...]} for the LAST run of >= min_len consecutive launches of each kernel."""
    runs, i = {}, 0
    while i < len(launches):
        j = i
        while j < len(launches) and launches[j]["kernel"] == launches[i]["kernel"]:
            j += 1
        op = op_of_kernel(launches[i]["kernel"])
        if op and j - i >= min_len:
            runs[op] = launches[i:j]
        i = j
    return runs


def summarise(path: str, workload: str, dtype: str, command: str):
    from . import streamops as so
    runs = op_major_runs(parse(path))
    kernels = {}
    for op, run in runs.items():
        body = run[1:]
        kernels[op] = {
            "kernel": run[0]["kernel"], "launches_in_run": len(run),
            "dram_read_bytes": round(statistics.median(l["dram__bytes_read.sum"] for l in body)),
            "dram_write_bytes": round(statistics.median(l["dram__bytes_write.sum"] for l in body)),
            "launch_us": round(statistics.median(l["gpu__time_duration.sum"] for l in body), 2),
            "tuning": so.get_tuning(op, dtype).as_dict(),
        }
    return {"workload": workload, "dtype": dtype, "region": "op-major (runs of one kernel), L2 state carried between launches",
            "command": command, "kernels": kernels}


def main(argv=None):
    p = argparse.ArgumentParser()
    p.add_argument("csv")
    p.add_argument("--workload", default="c2")
    p.add_argument("--dtype", default="f64")
    p.add_argument("--command", default="")
    p.add_argument("--out", default=None)
    args = p.parse_args(argv)
    from . import harness
    data = summarise(args.csv, args.workload, args.dtype, args.command)
    out = args.out or harness.traffic_file(args.workload)
    with open(out, "w") as f:
        f.write("# DRAM traffic per launch of each kernel, op-major region of bench.py, from one ncu capture.\n")
        f.write("# Written by `python -m paper_2510_00932_b200.ncu_summary`; bench.py reads `roofline.traffic` from here.\n")
        f.write(f"# Command: {args.command}\n")
        json.dump(data, f, indent=1)
        f.write("\n")
    for op, k in data["kernels"].items():
        print(f"{op:6s} read {k['dram_read_bytes'] / 1e6:8.1f} MB  write {k['dram_write_bytes'] / 1e6:8.1f} MB  {k['launch_us']:7.1f} us")
    return 0


if __name__ == "__main__":
    sys.exit(main())
