"""Size sweep of the five kernels (configuration 5): GB/s versus n across the L2-to-HBM transition.

    python -m paper_2510_00932_b200.sweep [--dtypes f64,f32] [--iters 20] [--out sweep.json] [--md sweep.md]
    python -m paper_2510_00932_b200.sweep --shapes [--iters 20] [--out shapes.json] [--md shapes.md]

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


def run_shapes(sizes=((1 << 25), (1 << 28)), iters=20, dtype="f64"):
    """Launch-shape sweep of the register-vector kernels (tuning kind 0): every combination of
    threads per block x vectors in flight per thread x grid form x cache-hint set, each timed
    op-major (`iters` launches in a row, one CUDA-event pair) on uniform [0,1) arrays, plus the
    time of one chain step (copy, scale, add, triad, dot) with the elementwise kernels or Dot set to
    that shape and everything else at its default. This is the sweep the defaults are chosen from.
    (Op-major launches do not consume their predecessor's output, so policies 7 and 8 store
    evict-first there, like 4; their two-phase stores show in the chain column.)"""
    import itertools
    import torch
    from . import harness, inputs
    from . import streamops as so

    if not torch.cuda.is_available():
        raise SystemExit("the sweep needs a CUDA device; there is no CPU fallback")
    so.lib()
    so.init(torch.cuda.current_device())
    stream = torch.cuda.current_stream()
    ew_shapes = [dict(threads=th, unroll=u, blocks_per_sm=bps, policy=pol)
                 for th, u, bps, pol in itertools.product((128, 256, 512), (1, 2, 4), (0, 4, 8), (4, 5, 7))]
    dot_shapes = [dict(threads=th, unroll=u, blocks_per_sm=bps, policy=pol, pipeline=pipe)
                  for pipe, th, u, bps, pol in itertools.product((0, 1), (256, 512), (1, 2, 4), (0, 1, 2, 3, 4), (0, 4))
                  if not (pipe == 1 and u == 1)]
    rows = []
    for n in sizes:
        w = inputs.sweep_workload(dtype, n)
        a, b, c = (torch.from_numpy(v).cuda() for v in inputs.make_arrays(w))
        d = torch.zeros(1, dtype=a.dtype, device="cuda")
        calls = {"copy": lambda: so.copy(a, c), "scale": lambda: so.scale(c, b, w.scalar),
                 "add": lambda: so.add(a, b, c), "triad": lambda: so.triad(b, c, a, w.scalar),
                 "dot": lambda: so.dot(a, b, d)}

        def time_it(f, count):
            for _ in range(3):
                f()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(count):
                f()
            e1.record(stream)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / count * 1e3

        def chain():
            for f in calls.values():
                f()

        so.reset_tuning()
        base = {op: time_it(f, iters) for op, f in calls.items()}
        rows.append({"n": n, "shape": "default", **{op: round(us, 2) for op, us in base.items()}, "chain_us": round(time_it(chain, iters), 2)})
        for group, ops, shapes in (("ew", so.OPS[:4], ew_shapes), ("dot", ("dot",), dot_shapes)):
            for shape in shapes:
                so.reset_tuning()
                for op in ops:
                    so.set_tuning(op, dtype, **shape)
                row = {"n": n, "shape": {"group": group, **shape}}
                for op in ops:
                    row[op] = round(time_it(calls[op], iters), 2)
                row["chain_us"] = round(time_it(chain, iters), 2)
                rows.append(row)
        so.reset_tuning()
        so.check()
        del a, b, c
    return rows


def shapes_markdown(rows) -> str:
    out = []
    for n in sorted({r["n"] for r in rows}):
        mine = [r for r in rows if r["n"] == n]
        base = mine[0]
        out.append(f"### n = {n} (fp64, {n * 8 / 2**20:.0f} MiB per array); microseconds per launch, op-major; chain = one step of the five kernels\n")
        out.append("default tuning: " + ", ".join(f"{op} {base[op]}" for op in ("copy", "scale", "add", "triad", "dot")) + f", chain {base['chain_us']}\n")
        for group, ops in (("ew", ("copy", "scale", "add", "triad")), ("dot", ("dot",))):
            out.append(("| kernel " if group == "dot" else "") + "| threads | unroll | grid | policy | " + " | ".join(ops) + " | chain step |")
            out.append(("|---" if group == "dot" else "") + "|---|---|---|---|" + "---|" * (len(ops) + 1))
            for r in mine[1:]:
                sh = r["shape"]
                if sh["group"] != group:
                    continue
                grid = "block per tile" if sh["blocks_per_sm"] == 0 and group == "ew" else ("automatic" if sh["blocks_per_sm"] == 0 else f"{sh['blocks_per_sm']} per SM")
                kern = ("| rolling slots " if sh.get("pipeline") else "| tiles ") if group == "dot" else ""
                out.append(kern + f"| {sh['threads']} | {sh['unroll']} | {grid} | {sh['policy']} | " + " | ".join(f"{r[o]:.1f}" for o in ops) + f" | {r['chain_us']:.1f} |")
            out.append("")
    return "\n".join(out) + "\n"


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
    p.add_argument("--shapes", action="store_true",
                   help="launch-shape sweep of the register-vector kernels at n = 2^25 and 2^28 instead of the size sweep")
    args = p.parse_args(argv)
    if args.shapes:
        rows = run_shapes(iters=args.iters)
        md = shapes_markdown(rows)
        if args.out:
            with open(args.out, "w") as f:
                json.dump(rows, f, indent=1)
        if args.md:
            with open(args.md, "w") as f:
                f.write(md)
        sys.stdout.write(md)
        return 0
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
