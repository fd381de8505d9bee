"""The five kernels over arrays that are split across GPUs, one process per GPU.

Copy, Mul (scale), Add and Triad are independent per index, so each rank runs the library's
kernels on its own contiguous piece of every array and nothing is exchanged. Dot needs one
exchange: every rank computes the double-precision partial dot product of its piece
(``stream_dot_f64`` / ``stream_dot_wide_f32``), the world's partial sums are all-gathered (8 bytes
per rank, NCCL between GPUs), and every rank adds them left to right in rank order
(``stream_fold_*``). The order is fixed, so all ranks hold the same bits and repeated calls repeat
them; an all-reduce, whose summation order is the library's business, would not promise that.

    python -m torch.distributed.run --nproc-per-node N -m paper_2510_00932_b200.sharded --n 33554432

runs the chain over N GPUs and prints the whole-array GB/s (strong scaling: n is the total length).
"""
from __future__ import annotations

import argparse
import json
import sys


def shard_bounds(n: int, world: int, rank: int, align: int = 1) -> tuple[int, int]:
    """[lo, hi) of rank's piece of n elements: contiguous, in rank order, covering 0..n exactly once,
    every boundary except n itself a multiple of `align` elements (so that every piece starts on the
    vector alignment of the whole array), sizes differing by at most one aligned block."""
    if not (world >= 1 and 0 <= rank < world and n >= 0 and align >= 1):
        raise ValueError("shard_bounds: need world >= 1, 0 <= rank < world, n >= 0, align >= 1")
    blocks = -(-n // align)                          # aligned blocks, the last one possibly short
    per, extra = divmod(blocks, world)
    lo_b = rank * per + min(rank, extra)
    hi_b = lo_b + per + (1 if rank < extra else 0)
    return min(lo_b * align, n), min(hi_b * align, n)


class ShardedStream:
    """One rank's view of the sharded kernels. `ops` supplies copy/scale/add/triad/dot_wide/fold
    on this rank's tensors (the CUDA binding by default); `gather(partial, gathered)` fills the
    `world`-element float64 tensor `gathered` with every rank's one-element `partial` in rank order
    (``torch.distributed.all_gather`` on `group` by default)."""

    def __init__(self, world: int, rank: int, device, ops=None, group=None, gather=None):
        import torch
        if ops is None:
            from . import streamops as ops           # the CUDA kernels; raises if the library is missing
        self.world, self.rank, self.ops, self.group = world, rank, ops, group
        self.partial = torch.zeros(1, dtype=torch.float64, device=device)
        self.gathered = torch.zeros(world, dtype=torch.float64, device=device)
        self._gather = gather or self._dist_gather

    def _dist_gather(self, partial, gathered):
        import torch.distributed as dist
        if self.world == 1:
            gathered.copy_(partial)
            return
        dist.all_gather([gathered[r:r + 1] for r in range(self.world)], partial, group=self.group)

    # the four elementwise kernels: purely local
    def copy(self, x, out):
        return self.ops.copy(x, out)

    def scale(self, x, out, scalar):
        return self.ops.scale(x, out, scalar)

    def add(self, x, y, out):
        return self.ops.add(x, y, out)

    def triad(self, x, y, out, scalar):
        return self.ops.triad(x, y, out, scalar)

    def dot(self, x, y, out):
        """out[0] = dot product of the WHOLE arrays (identical bits on every rank), from this
        rank's pieces x, y."""
        self.ops.dot_wide(x, y, self.partial)
        self._gather(self.partial, self.gathered)
        return self.ops.fold(self.gathered, out)

    def chain(self, a, b, c, dot_out, scalar):
        """c <- a; b <- s*c; c <- a+b; a <- b+s*c; dot_out <- dot(a, b) over the whole arrays."""
        self.copy(a, c)
        self.scale(c, b, scalar)
        self.add(a, b, c)
        self.triad(b, c, a, scalar)
        return self.dot(a, b, dot_out)


def main(argv=None):
    import torch
    import torch.distributed as dist
    from . import harness, inputs
    from . import streamops as so

    p = argparse.ArgumentParser()
    p.add_argument("--n", type=int, default=1 << 25)
    p.add_argument("--dtype", default="f64", choices=["f64", "f32"])
    p.add_argument("--steps", type=int, default=100)
    args = p.parse_args(argv)
    rank, local_rank, world = harness.dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("the sharded run needs CUDA devices; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    so.init(local_rank)
    w = inputs.sweep_workload(args.dtype, args.n)
    lo, hi = shard_bounds(args.n, world, rank, align=32 // w.itemsize)
    a, b, c = (torch.from_numpy(v[lo:hi].copy()).to(device) for v in inputs.make_arrays(w))
    out = torch.zeros(1, dtype=a.dtype, device=device)
    sh = ShardedStream(world, rank, device)
    for _ in range(5):
        sh.chain(a, b, c, out, w.scalar)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(device)
    e0.record()
    for _ in range(args.steps):
        sh.chain(a, b, c, out, w.scalar)
    e1.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(device)
    ms = harness.max_over_ranks(e0.elapsed_time(e1) / args.steps, device)
    if rank == 0:
        print(json.dumps({"n": args.n, "dtype": args.dtype, "n_gpus": world, "ms_per_step": round(ms, 5),
                          "gbs_whole_array": round(harness.step_bytes(args.n, w.itemsize) / ms / 1e6, 1),
                          "scaling": "strong", "dot": float(out.item())}))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
