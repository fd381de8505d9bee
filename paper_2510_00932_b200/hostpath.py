"""Host-overhead path at the paper's own problem sizes.

The paper ran the five kernels at ARRAY_SIZE 2000896 / 4000768 / 6000640 with num_times 100..300
(Table 1). At those sizes the arrays sit in L2, a kernel lasts a few microseconds, and what an
iteration costs is decided on the host: the edits the paper reports for these kernels (Table 2)
replaced a blocking copy by a synchronise, nothing else. This module measures the iteration
wall-clock of the same five-kernel pass under four host-side protocols:

  sync_each    five library calls, then a blocking read of the dot product, every iteration
  async_calls  five library calls per iteration, one synchronise at the end
  chain_call   one library call (streamops_chain_*) per iteration, one synchronise at the end
  graph        the pass captured once in a CUDA graph whose Dot writes its result straight into
               pinned (device-mapped) host memory; one graph launch per iteration, the result is
               picked up through an event, never through a copy

    python -m paper_2510_00932_b200.hostpath [--runs 10] [--out hostpath.json]
"""
from __future__ import annotations

import argparse
import json
import statistics
import sys
import time

PAPER_ARRAY_SIZES = (2000896, 4000768, 6000640)
PAPER_NUM_TIMES = (100, 200, 300)


class ChainGraph:
    """The five-kernel pass over (a, b, c), captured once and replayed with one launch per
    iteration. The Dot's output pointer is pinned host memory (device-accessible under unified
    addressing), so the result lands on the host without a copy node in the graph. The captured Dot
    uses one of the library's workspace slots reserved for graphs (never handed to ordinary calls),
    and the elementwise launches keep the traversal directions chosen at capture time; both are part
    of the graph. Replays of one ChainGraph must not overlap each other (they share that slot)."""

    def __init__(self, a, b, c, scalar: float):
        import torch
        from . import streamops as so
        self._torch = torch
        self.a, self.b, self.c, self.scalar = a, b, c, float(scalar)
        self.dot_host = torch.zeros(1, dtype=a.dtype).pin_memory()
        self.done = torch.cuda.Event()
        suf = so._suffix(a)
        fn = getattr(so.lib(), f"streamops_chain_{suf}")
        args = (a.data_ptr(), b.data_ptr(), c.data_ptr(), self.dot_host.data_ptr(), self.scalar, a.numel())

        def issue():
            so._raise(fn(*args, torch.cuda.current_stream(a.device).cuda_stream))

        so.init(a.get_device())                      # capture must not allocate
        issue()                                      # warm-up outside capture (module load, Dot slot)
        torch.cuda.synchronize(a.device)
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            issue()

    def replay(self):
        """Launches one pass; returns immediately."""
        self.graph.replay()
        self.done.record()

    def result(self):
        """Waits on the event of the last replay (no copy is issued) and returns the dot product."""
        self.done.synchronize()
        return self.dot_host.item()


def _arrays(dtype: str, n: int, seed: int = 4):
    import torch
    from . import inputs
    w = inputs.Workload("hostpath", dtype, n, "uniform01", seed, 0.4, 1)
    return w, [torch.from_numpy(v).cuda() for v in inputs.make_arrays(w)]


def time_protocols(dtype: str, n: int, num_times: int, runs: int = 10):
    """Wall-clock per iteration (microseconds, mean and standard deviation over `runs`) of the
    four protocols, each run starting from the same seeded arrays."""
    import torch
    from . import streamops as so
    w, (a0, b0, c0) = _arrays(dtype, n)
    a, b, c = a0.clone(), b0.clone(), c0.clone()
    dd = torch.zeros(1, dtype=a.dtype, device="cuda")
    graph = ChainGraph(a, b, c, w.scalar)

    def reset():
        a.copy_(a0); b.copy_(b0); c.copy_(c0)
        torch.cuda.synchronize()

    def five_calls():
        so.copy(a, c); so.scale(c, b, w.scalar); so.add(a, b, c); so.triad(b, c, a, w.scalar); so.dot(a, b, dd)

    def sync_each():
        for _ in range(num_times):
            five_calls()
            dd.item()

    def async_calls():
        for _ in range(num_times):
            five_calls()
        torch.cuda.synchronize()

    def chain_call():
        for _ in range(num_times):
            so.chain(a, b, c, dd, w.scalar)
        torch.cuda.synchronize()

    def graph_replay():
        for _ in range(num_times):
            graph.replay()
        graph.result()

    out = {}
    for name, fn in (("sync_each", sync_each), ("async_calls", async_calls), ("chain_call", chain_call),
                     ("graph", graph_replay)):
        per_iter = []
        for r in range(runs + 1):
            reset()
            t0 = time.perf_counter()
            fn()
            dt = time.perf_counter() - t0
            if r > 0:                                   # first run warms up
                per_iter.append(dt / num_times * 1e6)
        out[name] = {"us_per_iter": round(statistics.fmean(per_iter), 2),
                     "std": round(statistics.pstdev(per_iter), 2)}
    so.check()
    return out


def main(argv=None):
    p = argparse.ArgumentParser()
    p.add_argument("--runs", type=int, default=10)
    p.add_argument("--dtype", default="f64")
    p.add_argument("--out", default=None)
    args = p.parse_args(argv)
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device; there is no CPU fallback")
    rows = []
    print("| ARRAY_SIZE | num_times | sync_each µs/iter | async_calls | chain_call | graph | sync_each / graph |")
    print("|---|---|---|---|---|---|---|")
    for n in PAPER_ARRAY_SIZES:
        for nt in PAPER_NUM_TIMES:
            r = time_protocols(args.dtype, n, nt, args.runs)
            rows.append({"n": n, "num_times": nt, "dtype": args.dtype, **r})
            f = lambda k: f"{r[k]['us_per_iter']:.1f} ± {r[k]['std']:.1f}"
            print(f"| {n} | {nt} | {f('sync_each')} | {f('async_calls')} | {f('chain_call')} | {f('graph')} | "
                  f"{r['sync_each']['us_per_iter'] / r['graph']['us_per_iter']:.2f}× |", flush=True)
    if args.out:
        with open(args.out, "w") as fh:
            json.dump(rows, fh, indent=1)
    return 0


if __name__ == "__main__":
    sys.exit(main())
