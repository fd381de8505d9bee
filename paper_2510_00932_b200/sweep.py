"""Size sweep of the five kernels (configuration 5): GB/s versus n across the L2-to-HBM transition.

    python -m paper_2510_00932_b200.sweep [--dtypes f64,f32] [--iters 20] [--out sweep.json] [--md sweep.md]

For every size of ``inputs.SWEEP_SIZES`` (powers of two 2^16..2^29, 2^24+7 for the tail path, and
the three ARRAY_SIZE values of the paper's Table 1) and both element types, each kernel is
launched ``iters`` times back to back on seeded uniform [0,1) arrays and timed with one CUDA-event
pair; the report gives the mean time per launch and the algorithmic GB/s (2 arrays for
copy/scale/dot, 3 for add/triad). Sizes whose three arrays fit in L2 measure L2, not HBM: the
table says which is which.
"""
from __future__ import annotations

import argparse
import json
import sys

L2_BYTES = 126 * 1000 * 1000


def run(dtypes, iters, sizes=None):
    import torch
    from . import harness, inputs
    from . import streamops as so

    if not torch.cuda.is_available():
        raise SystemExit("the sweep needs a CUDA device; there is no CPU fallback")
    so.lib()
    so.init(torch.cuda.current_device())
    stream = torch.cuda.current_stream()
    rows = []
    for t in dtypes:
        for n in (sizes or inputs.SWEEP_SIZES):
            w = inputs.sweep_workload(t, n)
            a, b, c = (torch.from_numpy(v).cuda() for v in inputs.make_arrays(w))
            d = torch.zeros(1, dtype=a.dtype, device="cuda")
            calls = {"copy": lambda: so.copy(a, c), "scale": lambda: so.scale(c, b, w.scalar),
                     "add": lambda: so.add(a, b, c), "triad": lambda: so.triad(b, c, a, w.scalar),
                     "dot": lambda: so.dot(a, b, d)}
            row = {"dtype": t, "n": n, "array_bytes": n * w.itemsize,
                   "resident": "L2" if 3 * n * w.itemsize <= L2_BYTES else "HBM"}
            for op, f in calls.items():
                for _ in range(3):
                    f()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record(stream)
                for _ in range(iters):
                    f()
                e1.record(stream)
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / iters
                row[op] = {"us": round(ms * 1e3, 2), "gbs": round(harness.op_bytes(op, n, w.itemsize) / ms / 1e6, 1)}
            so.check()
            rows.append(row)
            del a, b, c
    return rows


def to_markdown(rows) -> str:
    ops = ("copy", "scale", "add", "triad", "dot")
    out = ["| dtype | n | array | resident | " + " | ".join(f"{o} GB/s" for o in ops) + " |",
           "|---|---|---|---|" + "---|" * len(ops)]
    for r in rows:
        size = r["array_bytes"]
        human = f"{size / 2**20:.1f} MiB" if size < 2**30 else f"{size / 2**30:.1f} GiB"
        out.append(f"| {r['dtype']} | {r['n']} | {human} | {r['resident']} | "
                   + " | ".join(f"{r[o]['gbs']:.0f}" for o in ops) + " |")
    return "\n".join(out) + "\n"


def main(argv=None):
    p = argparse.ArgumentParser()
    p.add_argument("--dtypes", default="f64,f32")
    p.add_argument("--iters", type=int, default=20)
    p.add_argument("--out", default=None)
    p.add_argument("--md", default=None)
    args = p.parse_args(argv)
    rows = run(args.dtypes.split(","), args.iters)
    md = to_markdown(rows)
    if args.out:
        with open(args.out, "w") as f:
            json.dump(rows, f, indent=1)
    if args.md:
        with open(args.md, "w") as f:
            f.write(md)
    sys.stdout.write(md)
    return 0


if __name__ == "__main__":
    sys.exit(main())
