"""The compensated Dot (tuning field `compensated`), through the C ABI: on inputs whose dot product
cancels by many orders of magnitude it stays within the usual tolerance of the exactly rounded
result where the plain Dot cannot, it agrees with the plain Dot on benign inputs, it visits every
index once, and it returns identical bits on every call."""
import numpy as np
import pytest

from paper_2510_00932_b200 import inputs

pytestmark = pytest.mark.gpu
TOL = {"f64": 1e-12, "f32": 1e-5}


@pytest.fixture(scope="module")
def so():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00932_b200 import streamops
    streamops.lib()
    yield streamops
    streamops.reset_tuning()


def _gpu_dot(so, x, y, **tuning):
    import torch
    t = "f64" if x.dtype == np.float64 else "f32"
    so.reset_tuning()
    so.set_tuning("dot", t, **tuning)
    dx, dy = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    out = torch.zeros(1, dtype=dx.dtype, device="cuda")
    so.dot(dx, dy, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()[0]


@pytest.mark.parametrize("log2_big,tol", [(30, 1e-12), (45, 1e-12), (60, 1e-9)])
def test_heavy_cancellation_against_the_exact_dot_product(so, oracle, log2_big, tol):
    # Dot2's error is about u + n^2 u^2 cond (u = 2^-53): inside 1e-12 up to cond ~ 2^46 at this n, and
    # still nine digits at cond ~ 2^61, where a plain double sum (n u cond) has no correct digit left
    from oracle import exact
    x, y = inputs.make_cancelling(99_999, "f64", seed=31, log2_big=log2_big)
    truth = float(exact.dot_exact_bigint(x, y))                 # exact rational value, rounded once
    cond = oracle.dot_abs(x, y) / abs(truth)
    assert cond > 2.0 ** log2_big
    got = _gpu_dot(so, x, y, compensated=1)
    assert abs(got - truth) <= tol * abs(truth), (got, truth, cond)
    if log2_big <= 45:
        assert abs(oracle.dot(x, y) - truth) <= tol * abs(truth)          # the oracle's own Dot2 agrees
    if log2_big >= 60:                                                    # the plain sum has lost everything here
        plain = _gpu_dot(so, x, y, compensated=0)
        assert abs(plain - truth) > 1e-3 * abs(truth)


@pytest.mark.parametrize("t,n", [("f64", (1 << 22) + 13), ("f32", (1 << 22) + 13), ("f64", 7), ("f32", 100_003)])
@pytest.mark.parametrize("shape", [dict(), dict(threads=128, unroll=1, blocks_per_sm=1), dict(threads=256, unroll=2, blocks_per_sm=8)])
def test_large_cancelling_and_benign_inputs_against_the_oracle(so, oracle, t, n, shape):
    x, y = inputs.make_cancelling(n, t, seed=32, log2_big=36 if t == "f64" else 20)
    want = oracle.dot(x, y)
    got = _gpu_dot(so, x, y, compensated=1, **shape)
    assert abs(float(got) - want) <= TOL[t] * abs(want) + (np.finfo(np.float32).eps * abs(want) if t == "f32" else 0)
    w = inputs.WORKLOADS["c1" if t == "f64" else "c3"]
    a, b, _ = inputs.make_arrays(w, n)
    want = oracle.dot(a, b)
    comp, plain = _gpu_dot(so, a, b, compensated=1, **shape), _gpu_dot(so, a, b, compensated=0, **shape)
    assert abs(float(comp) - want) <= TOL[t] * abs(want) and abs(float(plain) - want) <= TOL[t] * abs(want)


def test_every_index_once_unaligned_pointers_and_repeatability(so, oracle):
    import torch
    so.reset_tuning(); so.set_tuning("dot", "f64", compensated=1)
    n = (1 << 18) + 5
    x = inputs.make_arrays(inputs.WORKLOADS["c1"], n + 1)[0]
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    for off in (0, 1):                                           # 1: not 32-byte aligned -> scalar loop
        dx = torch.from_numpy(x).cuda()[off:off + n]
        for k in (0, 1, 31, 4095, 8192, n // 2, n - 6, n - 1):
            e = torch.zeros(n + 1, dtype=torch.float64, device="cuda")[off:off + n]
            e[k] = 1.0
            so.dot(dx, e, out)
            assert out.item() == x[off + k]
        bits = set()
        dy = torch.from_numpy(x[::-1].copy()).cuda()[off:off + n]
        for _ in range(10):
            so.dot(dx, dy, out)
            bits.add(out.cpu().numpy().tobytes())
        assert len(bits) == 1
    so.check()
