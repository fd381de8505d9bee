"""Behaviour of the C-ABI boundary under conditions the parity tests do not reach: more Dots in
flight than workspace slots, a Dot recorded into a CUDA graph while ordinary Dots run, a bounded
wait inside a bulk-copy kernel that runs out (on purpose: with a limit of a few attempts, so the
wait ends by itself at once), and the host-buffer entry point on arrays many times larger than its
ring of device buffers."""
import threading

import numpy as np
import pytest

from conftest import assert_bits_equal
from paper_2510_00932_b200 import inputs

pytestmark = pytest.mark.gpu
DOT_SLOTS, CAPTURE_SLOTS = 24, 8


@pytest.fixture(scope="module")
def torch():
    import torch as _torch
    if not _torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return _torch


@pytest.fixture()
def so(torch):
    from paper_2510_00932_b200 import streamops
    streamops.lib()
    streamops.reset_tuning()
    streamops.set_wait_limit(0)
    streamops.set_host_piece_mib(16)
    yield streamops
    streamops.reset_tuning()
    streamops.set_wait_limit(0)
    streamops.set_host_piece_mib(16)
    torch.cuda.synchronize()


def _uniform(t, n, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.random(n) if t == "f64" else rng.random(n, dtype=np.float32)


def test_more_dots_in_flight_than_slots_is_refused_never_wrong(so, torch, oracle):
    """40 Dots on 40 streams, all held back behind a few milliseconds of other work so that none can
    finish while they are being issued: the first 24 get a slot each, the others are refused with
    the workspace status and leave their output alone; every accepted one gives the oracle's value.
    After a synchronise every stream is served again."""
    L = so.lib()
    n = 1 << 24
    x = torch.from_numpy(_uniform("f64", n, 71)).cuda()
    ys = [torch.from_numpy(_uniform("f64", n, 72 + k)).cuda() for k in range(4)]
    want = [oracle.dot(x.cpu().numpy(), y.cpu().numpy()) for y in ys]
    streams = [torch.cuda.Stream() for _ in range(40)]
    outs = torch.full((40,), -7.0, dtype=torch.float64, device="cuda")
    big = torch.zeros(1 << 28, dtype=torch.float64, device="cuda")
    big2 = torch.empty_like(big)
    torch.cuda.synchronize()
    gate_stream, gate = torch.cuda.Stream(), torch.cuda.Event()
    with torch.cuda.stream(gate_stream):
        for _ in range(12):                                  # ~4 GB of traffic each: several milliseconds in all
            big2.copy_(big)
        gate.record()
    for s in streams:
        s.wait_event(gate)
    status = []
    for k, s in enumerate(streams):
        status.append(L.stream_dot_f64(x.data_ptr(), ys[k % 4].data_ptr(), outs[k:k + 1].data_ptr(), 0.0, n, s.cuda_stream))
    torch.cuda.synchronize()
    got = outs.cpu().numpy()
    # torch hands out streams from a pool, so some of the 40 share a handle: a stream that already
    # holds a slot is served again (its Dots run in order); a new stream beyond the 24th is refused
    owners, expect = set(), []
    for s in streams:
        if s.cuda_stream in owners or len(owners) < DOT_SLOTS:
            owners.add(s.cuda_stream)
            expect.append(0)
        else:
            expect.append(5)
    assert status == expect and 5 in status
    for k, st in enumerate(status):
        if st == 0:
            assert abs(got[k] - want[k % 4]) <= 1e-12 * abs(want[k % 4]), k
        else:
            assert got[k] == -7.0, k
    assert "slot" in so.status_string(5)
    # a refused call launched nothing; everything has drained now, so every stream gets a slot again
    for k, s in enumerate(streams):
        assert L.stream_dot_f64(x.data_ptr(), ys[k % 4].data_ptr(), outs[k:k + 1].data_ptr(), 0.0, 1 << 12, s.cuda_stream) == 0
        s.synchronize()


def test_one_stream_never_runs_out_of_slots(so, torch):
    L = so.lib()
    n = 1 << 22
    x = torch.ones(n, dtype=torch.float64, device="cuda")
    outs = torch.zeros(200, dtype=torch.float64, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    for k in range(200):                                     # 200 Dots queued on one stream: stream order, one slot
        assert L.stream_dot_f64(x.data_ptr(), x.data_ptr(), outs[k:k + 1].data_ptr(), 0.0, n - k, s) == 0
    torch.cuda.synchronize()
    assert (outs.cpu().numpy() == np.arange(n, n - 200, -1, dtype=np.float64)).all()


def test_captured_dot_keeps_its_own_slot_beside_live_calls(so, torch, oracle):
    """A graph whose Dot was captured replays while ordinary Dots run on other streams: both give
    the oracle's values (graph slots are never handed to ordinary calls)."""
    n = (1 << 22) + 5
    a, b = (torch.from_numpy(_uniform("f64", n, 81 + i)).cuda() for i in range(2))
    want = oracle.dot(a.cpu().numpy(), b.cpu().numpy())
    so.init(torch.cuda.current_device())
    dg = torch.zeros(1, dtype=torch.float64, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        so.dot(a, b, dg)                                      # warm-up outside capture
    side.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        so.dot(a, b, dg)
    live = [torch.cuda.Stream() for _ in range(6)]
    outs = torch.zeros(6, dtype=torch.float64, device="cuda")
    for rep in range(5):
        dg.zero_()
        torch.cuda.synchronize()
        g.replay()
        for k, s in enumerate(live):
            with torch.cuda.stream(s):
                so.dot(a, b, outs[k:k + 1])
        torch.cuda.synchronize()
        assert abs(dg.item() - want) <= 1e-12 * abs(want)
        assert all(abs(v - want) <= 1e-12 * abs(want) for v in outs.cpu().numpy())


@pytest.mark.parametrize("op", ["copy", "triad", "dot"])
def test_a_wait_that_runs_out_is_reported_once_and_the_library_carries_on(so, torch, oracle, op):
    """With a limit of one attempt (a probe that does not block) the first wait of a bulk-copy
    pipeline gives up before its data can have arrived. The kernel must flag it, let its copies in flight land, and return;
    streamops_check then reports the timeout exactly once, and ordinary calls are exact again."""
    L = so.lib()
    n = (1 << 21) + 13
    x, y = (_uniform("f64", n, 91 + i) for i in range(2))
    dx, dy = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    out = torch.zeros(n if op != "dot" else 1, dtype=torch.float64, device="cuda")
    so.check()                                              # flag clear to begin with
    so.set_tuning(op, "f64", kind=1, threads=128, blocks_per_sm=1, chunk_bytes=16384, stages=4)
    so.set_wait_limit(1)
    call = {"copy": lambda: so.copy(dx, out), "triad": lambda: so.triad(dx, dy, out, 0.4), "dot": lambda: so.dot(dx, dy, out)}[op]
    call()
    assert L.streamops_check(torch.cuda.current_stream().cuda_stream) == 6       # STREAMOPS_ERR_TIMEOUT
    assert "wait" in so.status_string(6)
    assert L.streamops_check(torch.cuda.current_stream().cuda_stream) == 0       # reported once
    # the default limit again: same pipeline, exact results; then the default kernels
    so.set_wait_limit(0)
    for _ in range(2):
        call()
        so.check()
        if op == "copy":
            assert_bits_equal(out.cpu().numpy(), x, "copy")
        elif op == "triad":
            assert_bits_equal(out.cpu().numpy(), oracle.triad(x, y, 0.4), "triad")
        else:
            w = oracle.dot(x, y)
            assert abs(out.item() - w) <= 1e-12 * abs(w)
        so.reset_tuning()


@pytest.mark.parametrize("t,scalar", [("f64", 0.4), ("f32", 3.0)])
def test_host_arrays_many_times_larger_than_the_device_ring(so, torch, oracle, t, scalar):
    """Pieces of 1 MiB make the ring 12 MiB of device memory; arrays of 40 MiB + a ragged end go
    round it ten times. Results are those of the oracle, and free device memory does not shrink
    with n once the ring exists."""
    so.set_host_piece_mib(1)
    itemsize = 8 if t == "f64" else 4
    n = (40 << 20) // itemsize + 1031
    a, b, c = (_uniform(t, n, 101 + i) for i in range(3))
    so.chain_host(*(v[:1000].copy() for v in (a, b, c)), scalar)        # creates the ring
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ha, hb, hc = a.copy(), b.copy(), c.copy()
    d = so.chain_host(ha, hb, hc, scalar)
    assert torch.cuda.mem_get_info()[0] == free_before
    oa, ob, oc, od = oracle.chain(a, b, c, scalar)
    assert_bits_equal(ha, oa, "a"); assert_bits_equal(hb, ob, "b"); assert_bits_equal(hc, oc, "c")
    assert abs(float(d) - od) <= (1e-12 if t == "f64" else 1e-5) * abs(od)
    # b and c are outputs only (the dataflow overwrites them before reading them): whatever they hold on
    # entry, NaN included, the results are the same
    ha, hb, hc = a.copy(), np.full_like(b, np.nan), np.full_like(c, np.nan)
    d2 = so.chain_host(ha, hb, hc, scalar)
    assert_bits_equal(ha, oa, "a"); assert_bits_equal(hb, ob, "b"); assert_bits_equal(hc, oc, "c")
    assert np.array([d2]).tobytes() == np.array([d]).tobytes()


def test_host_entry_point_from_two_threads(so, torch, oracle):
    so.set_host_piece_mib(2)
    n = (3 << 20) + 77
    sets = [[_uniform("f64", n, 111 + 3 * k + i) for i in range(3)] for k in range(2)]
    want = [oracle.chain(*s, 0.4) for s in sets]
    work = [[v.copy() for v in s] for s in sets]
    res = [None, None]
    dev = torch.cuda.current_device()

    def run(k):
        torch.cuda.set_device(dev)
        res[k] = so.chain_host(*work[k], 0.4)

    th = [threading.Thread(target=run, args=(k,)) for k in range(2)]
    for t in th:
        t.start()
    for t in th:
        t.join()
    for k in range(2):
        for got, w, name in zip(work[k], want[k][:3], "abc"):
            assert_bits_equal(got, w, f"thread {k}, {name}")
        assert abs(float(res[k]) - want[k][3]) <= 1e-12 * abs(want[k][3])


def test_binding_refuses_tensors_of_a_device_that_is_not_current(so, torch):
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two devices")
    x = torch.zeros(64, dtype=torch.float64, device="cuda:1")
    torch.cuda.set_device(0)
    with pytest.raises(ValueError):
        so.copy(x, x.clone())


def test_instrumented_dot_returns_the_ordinary_bits_and_ordered_time_stamps(so, torch):
    """stream_dot_timeline_f64 is the default fp64 Dot plus three timer readings per block: same bits
    as stream_dot_f64, stamps non-decreasing within a block, the finishing block the last to end."""
    n = (1 << 23) + 12
    rng = np.random.Generator(np.random.PCG64(131))
    x, y = (torch.from_numpy(rng.standard_normal(n)).cuda() for _ in range(2))
    out, ref = (torch.zeros(1, dtype=torch.float64, device="cuda") for _ in range(2))
    stamps = torch.zeros(3 * so.TIMELINE_MAX_BLOCKS, dtype=torch.int64, device="cuda")
    so.dot(x, y, ref)
    blocks = so.dot_timeline(x, y, out, stamps)
    torch.cuda.synchronize()
    assert out.cpu().numpy().tobytes() == ref.cpu().numpy().tobytes()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert blocks == 2 * sms
    t = stamps[:3 * blocks].cpu().numpy().reshape(blocks, 3)
    assert (t[:, 0] > 0).all() and (t[:, 0] <= t[:, 1]).all() and (t[:, 1] <= t[:, 2]).all()
    assert t[:, 2].max() - t[:, 0].min() < 5_000_000                      # a few hundred microseconds at most, in ns
    assert (stamps[3 * blocks:] == 0).all()
    L = so.lib()
    import ctypes
    b = ctypes.c_uint(0)
    assert L.stream_dot_timeline_f64(x[1:].data_ptr(), y[1:].data_ptr(), out.data_ptr(), n - 1, None, stamps.data_ptr(), ctypes.byref(b)) == 7
    assert L.stream_dot_timeline_f64(x.data_ptr(), y.data_ptr(), out.data_ptr(), n, None, None, ctypes.byref(b)) == 1
