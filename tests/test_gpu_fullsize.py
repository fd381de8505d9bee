"""Parity at the full sizes of the named configurations, in the launch configuration the
benchmark times (default tuning, one chain pass on device arrays), and closed-form checks at the
largest sweep sizes where byte offsets pass 2^32."""
import numpy as np
import pytest

from conftest import assert_bits_equal, bits
from paper_2510_00932_b200 import inputs

pytestmark = pytest.mark.gpu
DOT_TOL = {"f64": 1e-12, "f32": 1e-5}


@pytest.fixture(scope="module")
def so():
    import torch
    assert torch.cuda.is_available()
    from paper_2510_00932_b200 import streamops
    streamops.lib()
    streamops.reset_tuning()
    return streamops


def _independent_pass(so, torch, oracle, w, a, b, c):
    """Each kernel on the pristine seeded arrays (this is where random signs stress Dot)."""
    da, db, dc = (torch.from_numpy(v).cuda() for v in (a, b, c))
    out = torch.empty_like(da)
    dd = torch.zeros(1, dtype=da.dtype, device="cuda")
    so.copy(da, out); torch.cuda.synchronize()
    assert (bits(out.cpu().numpy()) == bits(a)).all(), "copy"
    so.scale(dc, out, w.scalar)
    assert_bits_equal(out.cpu().numpy(), oracle.scale(c, w.scalar), "scale")
    so.add(da, db, out)
    assert_bits_equal(out.cpu().numpy(), oracle.add(a, b), "add")
    so.triad(db, dc, out, w.scalar)
    assert_bits_equal(out.cpu().numpy(), oracle.triad(b, c, w.scalar), "triad")
    so.dot(da, db, dd)
    want = oracle.dot(a, b)
    mags = oracle.dot_abs(a, b)
    got = float(dd.item())
    assert abs(got - want) <= DOT_TOL[w.dtype] * abs(want), f"dot {got} vs {want} (kappa {mags / abs(want):.3g})"
    return mags / abs(want)


@pytest.mark.parametrize("name", ["c2", "c3"])
def test_full_size_configurations(so, oracle, name):
    import torch
    w = inputs.WORKLOADS[name]
    a, b, c = inputs.make_arrays(w)
    kappa = _independent_pass(so, torch, oracle, w, a, b, c)
    print(f"{name} condition number of the seeded dot {kappa:.3g}")
    # chain pass, as the benchmark runs it
    da, db, dc = (torch.from_numpy(v.copy()).cuda() for v in (a, b, c))
    dd = torch.zeros(1, dtype=da.dtype, device="cuda")
    so.chain(da, db, dc, dd, w.scalar)
    oa, ob, oc, od = oracle.chain(a, b, c, w.scalar)
    assert_bits_equal(da.cpu().numpy(), oa, "chain a")
    assert_bits_equal(db.cpu().numpy(), ob, "chain b")
    assert_bits_equal(dc.cpu().numpy(), oc, "chain c")
    assert abs(float(dd.item()) - od) <= DOT_TOL[w.dtype] * abs(od)
    so.check()


def test_largest_configuration_lognormal_signed(so, oracle):
    """n = 2^28 fp64 (2 GiB per array), log-normal magnitudes with random signs."""
    import torch
    w = inputs.WORKLOADS["c4"]
    a, b, c = inputs.make_arrays(w)
    kappa = _independent_pass(so, torch, oracle, w, a, b, c)
    print(f"c4 condition number {kappa:.3g}")
    so.check()


@pytest.mark.parametrize("t,logn", [("f64", 29), ("f32", 29)])
def test_largest_sweep_size_closed_forms(so, t, logn):
    """n = 2^29: byte offsets pass 2^32 (fp64: 4 GiB per array). Constants give known outputs, a
    ramp pins each index to its own value, unit vectors pin Dot's coverage at the far end."""
    import torch
    n = 1 << logn
    tdt = torch.float64 if t == "f64" else torch.float32
    npdt = np.float64 if t == "f64" else np.float32
    x = torch.arange(n, dtype=torch.int64, device="cuda").remainder_(1 << 20).to(tdt)   # exact small integers
    y = torch.full((n,), 0.5, dtype=tdt, device="cuda")
    out = torch.empty(n, dtype=tdt, device="cuda")
    probe = torch.tensor([0, 1, (1 << 20) + 3, n // 2 - 1, n // 2, n - (1 << 20) - 5, n - 2, n - 1], device="cuda")
    so.copy(x, out)
    assert torch.equal(out, x)
    so.scale(x, out, 0.25)
    assert torch.equal(out[probe], x[probe] * 0.25) and float(out.sum(dtype=torch.float64)) == float(x.sum(dtype=torch.float64)) * 0.25
    so.add(x, y, out)
    assert torch.equal(out[probe], x[probe] + 0.5) and torch.equal(out[-4096:], x[-4096:] + 0.5)
    so.triad(x, y, out, 4.0)
    assert torch.equal(out[probe], x[probe] + 2.0) and torch.equal(out[: 4096], x[: 4096] + 2.0)
    dd = torch.zeros(1, dtype=tdt, device="cuda")
    so.dot(y, y, dd)
    assert dd.item() == float(npdt(n * 0.25))
    e = torch.zeros(n, dtype=tdt, device="cuda")
    for k in (0, n // 2 + 12345, n - 1):
        e[k] = 1
        so.dot(x, e, dd)
        assert dd.item() == float(x[k].item()), k
        e[k] = 0
    so.check()


@pytest.mark.parametrize("t", ["f64", "f32"])
@pytest.mark.parametrize("n", [1 << 16, (1 << 24) + 7, 2000896, 4000768, 6000640])
def test_sweep_sizes_against_the_oracle(so, oracle, t, n):
    import torch
    w = inputs.sweep_workload(t, n)
    a, b, c = inputs.make_arrays(w)
    _independent_pass(so, torch, oracle, w, a, b, c)
