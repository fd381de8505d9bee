"""Timeline of one Dot launch inside a train of back-to-back launches (fp64, default kernel).

    python -m paper_2510_00932_b200.timeline [--n 33554432] [--train 20]

Launches `train` ordinary Dots, one instrumented Dot (stream_dot_timeline_f64: three global-timer stamps
per block) and `train` more, all on one stream with dependent-launch overlap as in normal use, and
prints, relative to the first block's start: when blocks start, when each block's data has all arrived,
when blocks end, and when the block that finishes the Dot is done; beside it the CUDA-event time per
launch of the whole train. The difference between "last data" and "finished" is what the reduction
costs after the memory system has gone idle.
"""
from __future__ import annotations

import argparse
import json
import sys


def percentiles(v):
    v = sorted(v)
    pick = lambda q: v[min(len(v) - 1, int(q * len(v)))]
    return {"min": v[0], "p10": pick(0.10), "p50": pick(0.50), "p90": pick(0.90), "p99": pick(0.99), "max": v[-1]}


def run(n: int, train: int):
    import torch
    from . import streamops as so

    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device; there is no CPU fallback")
    so.lib()
    so.init(torch.cuda.current_device())
    so.reset_tuning()
    x = torch.rand(n, dtype=torch.float64, device="cuda")
    y = torch.rand(n, dtype=torch.float64, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    ref = torch.zeros(1, dtype=torch.float64, device="cuda")
    stamps = torch.zeros(3 * so.TIMELINE_MAX_BLOCKS, dtype=torch.int64, device="cuda")
    stream = torch.cuda.current_stream()
    for _ in range(5):
        so.dot(x, y, ref)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(train):
        so.dot(x, y, ref)
    blocks = so.dot_timeline(x, y, out, stamps)
    for _ in range(train):
        so.dot(x, y, ref)
    e1.record(stream)
    torch.cuda.synchronize()
    assert out.item() == ref.item(), "the instrumented kernel must return the bits of the ordinary one"
    t = stamps[:3 * blocks].cpu().numpy().reshape(blocks, 3).astype("float64")
    t0 = t[:, 0].min()
    us = (t - t0) / 1e3
    finish = int(us[:, 2].argmax())
    return {"n": n, "blocks": blocks, "us_per_launch_of_the_train": round(e0.elapsed_time(e1) / (2 * train + 1) * 1e3, 2),
            "block_start_us": percentiles(us[:, 0].tolist()), "all_data_arrived_us": percentiles(us[:, 1].tolist()),
            "block_end_us": percentiles(us[:, 2].tolist()),
            "last_data_us": round(float(us[:, 1].max()), 2), "finished_us": round(float(us[:, 2].max()), 2),
            "finishing_block": finish, "after_last_data_us": round(float(us[:, 2].max() - us[:, 1].max()), 2),
            "bytes": 16 * n}


def main(argv=None):
    p = argparse.ArgumentParser()
    p.add_argument("--n", type=int, default=1 << 25)
    p.add_argument("--train", type=int, default=20)
    p.add_argument("--repeat", type=int, default=3)
    args = p.parse_args(argv)
    for _ in range(args.repeat):
        print(json.dumps(run(args.n, args.train)))
    return 0


if __name__ == "__main__":
    sys.exit(main())
