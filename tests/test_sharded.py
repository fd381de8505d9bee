"""The sharded form of the five kernels. On CPU: the partition arithmetic, and the whole exchange
path (local partial -> all-gather -> rank-ordered fold) over 2- and 3-rank gloo groups, with the
CPU oracle standing in for the per-rank kernels. On a GPU: the same path with the CUDA kernels and
the ranks of a 4-way split emulated one after the other on one device."""
import os
import socket

import numpy as np
import pytest

from paper_2510_00932_b200 import inputs
from paper_2510_00932_b200.sharded import ShardedStream, shard_bounds


@pytest.mark.parametrize("n,world,align", [(0, 3, 4), (1, 2, 4), (10, 4, 4), (1 << 20, 8, 4), ((1 << 20) + 7, 3, 8),
                                           (33, 5, 1), (100, 7, 16)])
def test_shard_bounds_partition_the_range(n, world, align):
    pieces = [shard_bounds(n, world, r, align) for r in range(world)]
    assert pieces[0][0] == 0 and pieces[-1][1] == n
    for (lo, hi), (lo2, _) in zip(pieces, pieces[1:] + [(n, n)]):
        assert lo <= hi == lo2                                  # contiguous, in rank order, no gaps
        assert lo % align == 0 or lo == n
    sizes = [hi - lo for lo, hi in pieces]
    assert max(sizes) - min(sizes) <= align + (align - 1)       # even up to one aligned block
    with pytest.raises(ValueError):
        shard_bounds(10, 2, 2)


class OracleOps:
    """The per-rank kernels, played by the CPU oracle on CPU torch tensors."""

    def __init__(self, oracle):
        self.o = oracle

    @staticmethod
    def _np(t):
        return t.numpy()

    def copy(self, x, out):
        out.numpy()[:] = self.o.copy(self._np(x))

    def scale(self, x, out, s):
        out.numpy()[:] = self.o.scale(self._np(x), s)

    def add(self, x, y, out):
        out.numpy()[:] = self.o.add(self._np(x), self._np(y))

    def triad(self, x, y, out, s):
        out.numpy()[:] = self.o.triad(self._np(x), self._np(y), s)

    def dot_wide(self, x, y, out64):
        out64[0] = self.o.dot(self._np(x), self._np(y)) if x.numel() else 0.0

    def fold(self, partials, out):
        out[0] = self.o.fold(self._np(partials))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n, dtype, out):
    import torch
    import torch.distributed as dist
    import oracle
    oracle.build()
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = inputs.sweep_workload(dtype, n)
        full = inputs.make_arrays(w)
        lo, hi = shard_bounds(n, world, rank, align=32 // w.itemsize)
        a, b, c = (torch.from_numpy(v[lo:hi].copy()) for v in full)
        res = torch.zeros(1, dtype=a.dtype)
        sh = ShardedStream(world, rank, "cpu", ops=OracleOps(oracle))
        sh.chain(a, b, c, res, w.scalar)
        out.put((rank, lo, hi, a.numpy().tobytes(), b.numpy().tobytes(), c.numpy().tobytes(),
                 res.numpy().tobytes(), sh.gathered.numpy().tobytes()))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,n,dtype", [(2, (1 << 16) + 5, "f64"), (3, 50001, "f32"), (2, 3, "f64")])
def test_gloo_ranks_reproduce_the_unsharded_oracle(oracle, world, n, dtype):
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q, port = ctx.Queue(), _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, n, dtype, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    w = inputs.sweep_workload(dtype, n)
    oa, ob, oc, od = oracle.chain(*inputs.make_arrays(w), w.scalar)
    np_t = np.float64 if dtype == "f64" else np.float32
    partials = []
    for rank, lo, hi, a, b, c, res, gathered in got:
        # elementwise results: bit for bit the matching piece of the unsharded oracle
        assert a == oa[lo:hi].tobytes() and b == ob[lo:hi].tobytes() and c == oc[lo:hi].tobytes()
        partials.append(oracle.dot(oa[lo:hi], ob[lo:hi]) if hi > lo else 0.0)
    want_gathered = np.array(partials, dtype=np.float64)
    want = np_t(oracle.fold(want_gathered))
    for rank, lo, hi, a, b, c, res, gathered in got:
        assert gathered == want_gathered.tobytes()              # every rank holds all partials in rank order
        assert res == np.array([want]).tobytes()                # and therefore the same bits
    tol = 1e-12 if dtype == "f64" else 1e-5
    assert abs(float(want) - od) <= tol * abs(od)               # and they are the whole arrays' dot product


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,n", [("f64", (1 << 22) + 13), ("f32", (1 << 22) + 13), ("f64", 5)])
def test_cuda_kernels_with_four_emulated_ranks(oracle, dtype, n):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00932_b200 import streamops as so
    so.lib(); so.reset_tuning()
    world = 4
    w = inputs.sweep_workload(dtype, n)
    full = inputs.make_arrays(w)
    dev = [torch.from_numpy(v).cuda() for v in full]
    bounds = [shard_bounds(n, world, r, align=32 // w.itemsize) for r in range(world)]
    board = torch.zeros(world, dtype=torch.float64, device="cuda")     # stands in for the all-gather

    def make_gather(rank):
        def gather(partial, gathered):
            board[rank:rank + 1].copy_(partial)
            gathered.copy_(board)
        return gather

    ranks = [ShardedStream(world, r, "cuda", gather=make_gather(r)) for r in range(world)]
    outs = [torch.zeros(1, dtype=dev[0].dtype, device="cuda") for _ in range(world)]
    views = [[d[lo:hi] for d in dev] for lo, hi in bounds]
    for sh, (a, b, c) in zip(ranks, views):                            # elementwise part, rank by rank
        sh.copy(a, c); sh.scale(c, b, w.scalar); sh.add(a, b, c); sh.triad(b, c, a, w.scalar)
    for sh, (a, b, c) in zip(ranks, views):                            # every rank posts its partial sum ...
        sh.ops.dot_wide(a, b, sh.partial); board[sh.rank:sh.rank + 1].copy_(sh.partial)
    for sh, (a, b, c), out in zip(ranks, views, outs):                 # ... then every rank runs the full dot
        sh.dot(a, b, out)
    torch.cuda.synchronize(); so.check()
    oa, ob, oc, od = oracle.chain(*full, w.scalar)
    U = np.uint64 if dtype == "f64" else np.uint32
    for got, want in zip(dev, (oa, ob, oc)):
        assert (got.cpu().numpy().view(U) == want.view(U)).all()
    results = {o.cpu().numpy().tobytes() for o in outs}
    assert len(results) == 1                                           # identical bits on every rank
    got = float(outs[0].item())
    tol = 1e-12 if dtype == "f64" else 1e-5
    assert abs(got - od) <= tol * abs(od)
    # the fold is the oracle's left-to-right sum of the gathered partials, bit for bit
    np_t = np.float64 if dtype == "f64" else np.float32
    assert np_t(oracle.fold(board.cpu().numpy())) == outs[0].cpu().numpy()[0]
    for r, (lo, hi) in enumerate(bounds):                              # each partial is within tolerance of its piece
        piece = oracle.dot(oa[lo:hi], ob[lo:hi]) if hi > lo else 0.0
        assert abs(float(board[r].item()) - piece) <= 1e-12 * max(abs(piece), 1e-300)


@pytest.mark.gpu
def test_fold_and_wide_dot_through_the_abi(oracle):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00932_b200 import streamops as so
    so.lib(); so.reset_tuning()
    rng = np.random.Generator(np.random.PCG64(78))
    cases = [np.array([1e16, 1.0, -1e16]), np.array([2.0 ** 53, 1.0, 1.0]), np.array([1.0, 1.0, 2.0 ** 53]),
             np.zeros(0), np.array([-0.0]), rng.standard_normal(1000) * np.exp(rng.uniform(-30, 30, 1000))]
    for p in cases:
        dp = torch.from_numpy(p.astype(np.float64)).cuda()
        o64 = torch.full((1,), 7.0, dtype=torch.float64, device="cuda")
        o32 = torch.full((1,), 7.0, dtype=torch.float32, device="cuda")
        so.fold(dp, o64); so.fold(dp, o32)
        want = oracle.fold(p.astype(np.float64))
        assert o64.cpu().numpy().tobytes() == np.array([want]).tobytes()
        assert o32.cpu().numpy().tobytes() == np.array([np.float32(want)]).tobytes()
    # the wide Dot of float arrays keeps what the float result rounds away
    w = inputs.WORKLOADS["c3"]
    a, b, _ = inputs.make_arrays(w, (1 << 20) + 3)
    da, db = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    wide = torch.zeros(1, dtype=torch.float64, device="cuda")
    narrow = torch.zeros(1, dtype=torch.float32, device="cuda")
    so.dot_wide(da, db, wide); so.dot(da, db, narrow)
    torch.cuda.synchronize()
    want, scale = oracle.dot(a, b), oracle.dot_abs(a, b)
    assert abs(wide.item() - want) <= 1e-13 * scale
    assert np.float32(wide.item()) == narrow.cpu().numpy()[0] or abs(narrow.item() - want) <= 1e-5 * abs(want)
    L = so.lib()
    assert L.stream_fold_f64(None, None, 0.0, 0, None) == 1 and L.stream_fold_f64(wide.data_ptr(), wide.data_ptr(), 0.0, 1, None) == 3
    assert L.stream_dot_wide_f32(da.data_ptr(), db.data_ptr(), wide.data_ptr() + 4, 0.0, 8, None) == 2
