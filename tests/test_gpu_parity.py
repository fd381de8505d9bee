"""Parity of the CUDA path against the CPU oracle, element by element, through the C ABI.

Elementwise kernels: bit-exact. Dot: relative 1e-12 (fp64) / 1e-5 (fp32) against the
compensated oracle, and bitwise repeatable. Sizes span several tiles and ragged tails; every
case runs under the default launch shape and a set of alternative ones (both vector widths,
every unroll, every cache-hint set, both tile orders, the bulk-copy pipelines)."""
import ctypes

import numpy as np
import pytest

from conftest import assert_bits_equal, bits
from gpu_util import BULK_TUNINGS, VEC_TUNINGS, Guarded
from paper_2510_00932_b200 import inputs

pytestmark = pytest.mark.gpu

TAILS = [0, 1, 2, 3, 4, 5, 7, 8, 15, 16, 17, 31, 32, 33, 1023, 1025]
DOT_TOL = {"f64": 1e-12, "f32": 1e-5}
ELEMENTWISE = ("copy", "scale", "add", "triad")


@pytest.fixture(scope="module")
def torch():
    import torch as _torch
    assert _torch.cuda.is_available(), "the gpu tests need a CUDA device"
    return _torch


@pytest.fixture(scope="module")
def so(torch):
    from paper_2510_00932_b200 import streamops
    streamops.lib()                      # raises if the CUDA library is not built
    streamops.init(0)
    yield streamops
    streamops.reset_tuning()


@pytest.fixture(autouse=True)
def _default_tuning(so):
    so.reset_tuning()
    yield
    so.check()                           # no bounded wait may have given up
    so.reset_tuning()


def _npdt(t):
    return np.float64 if t == "f64" else np.float32


def _data(t, n, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    mag = np.exp2(rng.integers(-10, 10, size=n).astype(np.float64))
    return ((2.0 * rng.random(n) - 1.0) * mag).astype(_npdt(t))


def _run_elementwise(so, torch, op, x, y, scalar, off=(0, 0, 0)):
    gx = Guarded(torch, host=x, offset=off[0])
    gy = Guarded(torch, host=y, offset=off[1])
    go = Guarded(torch, n=x.size, dtype=x.dtype, offset=off[2])
    if op == "copy":
        so.copy(gx.t, go.t)
    elif op == "scale":
        so.scale(gx.t, go.t, scalar)
    elif op == "add":
        so.add(gx.t, gy.t, go.t)
    else:
        so.triad(gx.t, gy.t, go.t, scalar)
    torch.cuda.synchronize()
    assert go.guards_intact() and gx.guards_intact() and gy.guards_intact(), "guard region overwritten"
    assert (bits(gx.host()) == bits(x)).all(), "input modified"
    return go.host()


def _oracle_elementwise(oracle, op, x, y, scalar):
    return {"copy": lambda: oracle.copy(x), "scale": lambda: oracle.scale(x, scalar),
            "add": lambda: oracle.add(x, y), "triad": lambda: oracle.triad(x, y, scalar)}[op]()


def _set_all(so, t, **fields):
    for op in so.OPS:
        so.set_tuning(op, t, **fields)


def _check_elementwise(so, torch, oracle, t, n, scalar, seed, off=(0, 0, 0)):
    x, y = _data(t, n, seed), _data(t, n, seed + 1)
    for op in ELEMENTWISE:
        got = _run_elementwise(so, torch, op, x, y, scalar, off)
        want = _oracle_elementwise(oracle, op, x, y, scalar)
        if op == "copy":
            assert (bits(got) == bits(want)).all(), f"copy {t} n={n} off={off}"
        else:
            assert_bits_equal(got, want, f"{op} {t} n={n} off={off}")


# ------------------------------------------------------------------ elementwise, default tuning
@pytest.mark.parametrize("t", ["f64", "f32"])
def test_tails_and_pointer_offsets(so, torch, oracle, t):
    """Every tail length, with the arrays starting 0..3 elements past an aligned address (so the
    32-byte, 16-byte and scalar kernels are all reached)."""
    scalar = 0.4 if t == "f64" else 3.0
    for n in TAILS:
        for off in [(0, 0, 0), (1, 1, 1), (2, 2, 2), (3, 3, 3), (0, 1, 2), (4, 0, 2), (2, 4, 0)]:
            _check_elementwise(so, torch, oracle, t, n, scalar, 1000 + n, off)


@pytest.mark.parametrize("t", ["f64", "f32"])
@pytest.mark.parametrize("n", [(1 << 20) + 7, 2000896, 3 * 148 * 512 * 8 + 4099])
def test_several_tiles_default_tuning(so, torch, oracle, t, n):
    _check_elementwise(so, torch, oracle, t, n, 0.4, 7)


@pytest.mark.parametrize("t", ["f64", "f32"])
@pytest.mark.parametrize("tuning", VEC_TUNINGS + BULK_TUNINGS, ids=lambda d: "-".join(f"{k[:3]}{v}" for k, v in d.items()))
def test_every_launch_shape(so, torch, oracle, t, tuning):
    _set_all(so, t, **tuning)
    for n in (0, 5, 1025, 300_007, (1 << 21) + 13):
        _check_elementwise(so, torch, oracle, t, n, 0.4, 11 + n)
    # offsets that leave only 16-byte or element alignment
    _check_elementwise(so, torch, oracle, t, 70_001, 3.0, 5, off=(2, 2, 2))
    _check_elementwise(so, torch, oracle, t, 70_001, 3.0, 6, off=(1, 3, 1))


@pytest.mark.parametrize("t", ["f64", "f32"])
def test_special_values(so, torch, oracle, t):
    sp = inputs.special_values(t)
    rng = np.random.Generator(np.random.PCG64(3))
    x = np.tile(sp, 40)
    y = rng.permutation(np.tile(sp, 40))
    snan = (np.array([0x7FF0000000000001], np.uint64).view(np.float64) if t == "f64"
            else np.array([0x7F800001], np.uint32).view(np.float32))
    xc = np.concatenate([x, snan])
    for tuning in [dict(kind=0), dict(kind=1)]:
        _set_all(so, t, **tuning)
        got = _run_elementwise(so, torch, "copy", xc, xc, 0.0)
        assert (bits(got) == bits(xc)).all(), "copy preserves every bit pattern"
        for op in ("scale", "add", "triad"):
            for s in (0.4, -3.0, 0.0):
                assert_bits_equal(_run_elementwise(so, torch, op, x, y, s),
                                  _oracle_elementwise(oracle, op, x, y, s), f"{op} specials s={s}")


@pytest.mark.parametrize("t", ["f64", "f32"])
def test_triad_takes_two_roundings_on_the_gpu(so, torch, oracle, t):
    from oracle import exact
    x, y = _data(t, 600, 13), _data(t, 600, 14)
    two, one = exact.triad_exact(x, y, 0.4), exact.fma_exact(x, y, 0.4)
    assert (bits(two) != bits(one)).sum() >= 20
    for tuning in [dict(kind=0), dict(kind=1)]:
        _set_all(so, t, **tuning)
        assert_bits_equal(_run_elementwise(so, torch, "triad", x, y, 0.4), two, "triad is mul then add")


@pytest.mark.parametrize("t", ["f64", "f32"])
def test_in_place(so, torch, oracle, t):
    n = 200_003
    x, y = _data(t, n, 21), _data(t, n, 22)
    for tuning in [dict(kind=0, policy=0), dict(kind=0, policy=1), dict(kind=0, policy=4), dict(kind=1)]:
        _set_all(so, t, **tuning)
        gx = Guarded(torch, host=x); so.scale(gx.t, gx.t, 0.4)
        assert_bits_equal(gx.host(), oracle.scale(x, 0.4), "scale in place")
        gx, gy = Guarded(torch, host=x), Guarded(torch, host=y); so.add(gx.t, gy.t, gx.t)
        assert_bits_equal(gx.host(), oracle.add(x, y), "add into x")
        gx, gy = Guarded(torch, host=x), Guarded(torch, host=y); so.triad(gx.t, gy.t, gy.t, 0.4)
        assert_bits_equal(gy.host(), oracle.triad(x, y, 0.4), "triad into y")
        assert gx.guards_intact() and gy.guards_intact()


# ------------------------------------------------------------------ dot
def _dot(so, torch, x, y, off=(0, 0)):
    gx, gy = Guarded(torch, host=x, offset=off[0]), Guarded(torch, host=y, offset=off[1])
    go = Guarded(torch, n=1, dtype=x.dtype)
    so.dot(gx.t, gy.t, go.t)
    torch.cuda.synchronize()
    assert go.guards_intact()
    return go.host()[0]


def _assert_dot_close(oracle, got, x, y, t, what=""):
    want = oracle.dot(x, y)
    denom = abs(want) if want != 0 else oracle.dot_abs(x, y)
    if t == "f32":
        # the output type is float: compare after the oracle's single rounding to float too
        assert abs(float(got) - want) <= DOT_TOL[t] * denom + 0.0, f"{what}: {got} vs {want}"
    else:
        assert abs(float(got) - want) <= DOT_TOL[t] * denom, f"{what}: {got} vs {want}"


@pytest.mark.parametrize("t", ["f64", "f32"])
@pytest.mark.parametrize("tuning", [dict()] + VEC_TUNINGS + BULK_TUNINGS + [dict(kind=0, two_pass=1)],
                         ids=lambda d: "-".join(f"{k[:3]}{v}" for k, v in d.items()) or "default")
def test_dot_matches_the_compensated_oracle(so, torch, oracle, t, tuning):
    so.set_tuning("dot", t, **tuning)
    for n in TAILS + [70_001, (1 << 20) + 7, (1 << 22) + 4099]:
        x, y = _data(t, n, 31 + n), _data(t, n, 32 + n)
        got = _dot(so, torch, x, y)
        if n == 0:
            assert got == 0 and not np.signbit(got)
        else:
            _assert_dot_close(oracle, got, x, y, t, f"dot n={n}")
    x, y = _data(t, 70_001, 41), _data(t, 70_001, 42)
    for off in [(1, 1), (2, 2), (3, 1), (0, 2)]:
        _assert_dot_close(oracle, _dot(so, torch, x, y, off), x, y, t, f"dot off={off}")


@pytest.mark.parametrize("t", ["f64", "f32"])
@pytest.mark.parametrize("tuning", [dict(), dict(kind=0, vec_bytes=16, unroll=4, threads=128, blocks_per_sm=1), dict(kind=1),
                                    dict(kind=0, pipeline=0, unroll=4, blocks_per_sm=0), dict(kind=0, pipeline=1, unroll=2, blocks_per_sm=0),
                                    dict(kind=0, pipeline=1, unroll=4, threads=256, blocks_per_sm=3)],
                         ids=["default", "vec16", "bulk", "tiles", "roll2", "roll4"])
def test_dot_visits_every_index_exactly_once(so, torch, oracle, t, tuning):
    """dot(x, e_k) = x_k exactly, for k in the tail, at tile and block boundaries: no index is
    skipped and none is counted twice (dot(x, 1) on integers would double-count otherwise)."""
    so.set_tuning("dot", t, **tuning)
    n = 148 * 2 * 512 * 8 + 2 * 4096 + 5        # a few full tiles per block plus a ragged end
    x = _data(t, n, 51)
    gx = Guarded(torch, host=x)
    e = torch.zeros(n, dtype=gx.t.dtype, device="cuda")
    out = torch.zeros(1, dtype=gx.t.dtype, device="cuda")
    ks = [0, 1, 3, 4, 7, 8, 511, 512, 4095, 4096, 8191, 8192, 148 * 4096 - 1, 148 * 4096, n // 2,
          n - 4101, n - 10, n - 6, n - 5, n - 4, n - 3, n - 2, n - 1]
    for k in ks:
        e[k] = 1
        so.dot(gx.t, e, out)
        assert out.item() == float(x[k]), f"k={k}"
        e[k] = 0
    # integers: the sum is exact in double, so any double-counting shows
    ones = torch.ones(n, dtype=gx.t.dtype, device="cuda")
    so.dot(ones, ones, out)
    assert out.item() == float(_npdt(t)(n))


@pytest.mark.parametrize("t", ["f64", "f32"])
@pytest.mark.parametrize("shape", [dict(unroll=2, threads=512, blocks_per_sm=0), dict(unroll=4, threads=256, blocks_per_sm=1),
                                   dict(unroll=2, threads=128, blocks_per_sm=2)], ids=["2x512", "4x256", "2x128"])
def test_rolling_slot_dot_counts_every_element_around_its_round_boundaries(so, torch, t, shape):
    """dot(1, 1) = n exactly (every partial sum is an integer below 2^53) for n just below, on and just
    above a tile, one pass of all blocks, one round of all slots and two rounds, plus a ragged end: a
    slot that skipped its last reload, or a tile counted by two slots, changes the count."""
    so.set_tuning("dot", t, pipeline=1, vec_bytes=32, kind=0, **shape)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    epv = 4 if t == "f64" else 8
    tile = shape["threads"] * epv
    grid = (shape["blocks_per_sm"] or 2) * sms
    marks = [tile, grid * tile, shape["unroll"] * grid * tile, 2 * shape["unroll"] * grid * tile]
    sizes = sorted({m + d for m in marks for d in (-tile - 1, -1, 0, 1, epv, tile - 1, tile + 3)} | {1, 5, epv, 3 * marks[2] + 2 * tile + 7})
    biggest = max(sizes)
    ones = torch.ones(biggest, dtype=torch.float64 if t == "f64" else torch.float32, device="cuda")
    out = torch.zeros(1, dtype=ones.dtype, device="cuda")
    for n in sizes:
        if n <= 0 or (t == "f32" and n > (1 << 24)):        # float holds integers exactly only up to 2^24
            continue
        so.dot(ones[:n], ones[:n], out)
        assert out.item() == float(n), f"n={n}"


def test_dot_f32_output_is_rounded_to_float(so, torch):
    n = (1 << 24) + 7
    ones = torch.ones(n, dtype=torch.float32, device="cuda")
    out = torch.zeros(1, dtype=torch.float32, device="cuda")
    so.dot(ones, ones, out)
    assert out.item() == 16777224.0


@pytest.mark.parametrize("t", ["f64", "f32"])
def test_dot_is_bitwise_repeatable(so, torch, t):
    n = (1 << 22) + 77
    w = inputs.Workload("det", t, n, "lognormal_signed" if t == "f64" else "uniform_pm1", 5, 0.4, 1)
    a, b, c = inputs.make_arrays(w)
    da, db, dc = (torch.from_numpy(v).cuda() for v in (a, b, c))
    streams = [torch.cuda.Stream() for _ in range(3)]
    outs = [torch.zeros(1, dtype=da.dtype, device="cuda") for _ in range(24)]
    torch.cuda.synchronize()
    for i, o in enumerate(outs):
        with torch.cuda.stream(streams[i % 3]):
            if i % 4 == 1:
                so.add(da, db, dc)                  # other kernels interleaved
            so.dot(da, db, o)
    torch.cuda.synchronize()
    ref = bits(outs[0].cpu().numpy())[0]
    assert all(bits(o.cpu().numpy())[0] == ref for o in outs)
    # a tuning round trip gives the same bits again
    base = so.get_tuning("dot", t).as_dict()
    so.set_tuning("dot", t, vec_bytes=16, unroll=4, threads=128)
    so.dot(da, db, outs[1])
    so.set_tuning("dot", t, **base)
    so.dot(da, db, outs[2])
    torch.cuda.synchronize()
    assert bits(outs[2].cpu().numpy())[0] == ref
    # the two-launch form sums in the same order as the single-launch form
    so.set_tuning("dot", t, two_pass=1)
    so.dot(da, db, outs[3])
    torch.cuda.synchronize()
    assert bits(outs[3].cpu().numpy())[0] == ref


# ------------------------------------------------------------------ chain and host entry
@pytest.mark.parametrize("name", ["c1"])
def test_chain_on_the_small_configuration(so, torch, oracle, name):
    w = inputs.WORKLOADS[name]
    a, b, c = inputs.make_arrays(w)
    da, db, dc = (torch.from_numpy(v.copy()).cuda() for v in (a, b, c))
    dd = torch.zeros(1, dtype=da.dtype, device="cuda")
    oa, ob, oc = a, b, c
    for _ in range(3):
        so.chain(da, db, dc, dd, w.scalar)
        oa, ob, oc, od = oracle.chain(oa, ob, oc, w.scalar)
        assert_bits_equal(da.cpu().numpy(), oa, "a"); assert_bits_equal(db.cpu().numpy(), ob, "b")
        assert_bits_equal(dc.cpu().numpy(), oc, "c")
        assert abs(dd.item() - od) <= DOT_TOL[w.dtype] * abs(od)


@pytest.mark.parametrize("n", [(1 << 20) + 3, 5 * (1 << 22) + 77])     # one piece; several 16 MiB pieces and a ragged last one
@pytest.mark.parametrize("t,scalar", [("f64", 0.4), ("f32", 3.0)])
def test_host_entry_point(so, torch, oracle, t, scalar, n):
    a, b, c = (_data(t, n, s) for s in (61, 62, 63))
    ha, hb, hc = a.copy(), b.copy(), c.copy()
    d = so.chain_host(ha, hb, hc, scalar)
    oa, ob, oc, od = oracle.chain(a, b, c, scalar)
    assert_bits_equal(ha, oa, "a"); assert_bits_equal(hb, ob, "b"); assert_bits_equal(hc, oc, "c")
    assert abs(float(d) - od) <= DOT_TOL[t] * abs(od)
    ha2, hb2, hc2 = a.copy(), b.copy(), c.copy()                        # pinned or not, first call or not: same bits
    pin = [torch.from_numpy(v).pin_memory() for v in (ha2, hb2, hc2)]
    d2 = so.chain_host(*(p.numpy() for p in pin), scalar)
    assert np.array([d2]).tobytes() == np.array([d]).tobytes()
    assert_bits_equal(pin[0].numpy(), oa, "a, pinned")
    assert so.chain_host(ha[:0], hb[:0], hc[:0], scalar) == 0


# ------------------------------------------------------------------ argument checks (host side)
def test_argument_errors(so, torch):
    L = so.lib()
    x = torch.zeros(1024, dtype=torch.float64, device="cuda")
    y = torch.zeros(1024, dtype=torch.float64, device="cuda")
    p, q = x.data_ptr(), y.data_ptr()
    assert L.stream_copy_f64(None, q, 0.0, 8, None) == 1
    assert L.stream_add_f64(p, None, q, 0.0, 8, None) == 1
    assert L.stream_copy_f64(None, None, 0.0, 0, None) == 0          # n = 0 touches nothing
    assert L.stream_dot_f64(None, None, None, 0.0, 0, None) == 1     # Dot always writes out
    assert L.stream_copy_f64(p + 4, q, 0.0, 8, None) == 2
    assert L.stream_scale_f32(p + 2, q, 0.0, 8, None) == 2
    assert L.stream_copy_f64(p, p + 8, 0.0, 100, None) == 3          # partial overlap
    assert L.stream_triad_f64(p, q, q + 512, 0.4, 100, None) == 3
    assert L.stream_scale_f64(p, p, 0.4, 100, None) == 0             # exact alias is allowed
    assert L.stream_dot_f64(p, q, p + 8 * 5, 0.0, 100, None) == 3    # Dot's out inside an input
    assert L.stream_dot_f64(p, q, p + 8 * 100, 0.0, 100, None) == 0
    t = so.Tuning()
    assert L.streamops_get_tuning(0, 1, ctypes.byref(t)) == 0
    t.unroll = 3
    assert L.streamops_set_tuning(0, 1, ctypes.byref(t)) == 7
    assert L.streamops_set_tuning(9, 1, ctypes.byref(t)) == 7
    torch.cuda.synchronize()
    assert so.launch_count() > 0
