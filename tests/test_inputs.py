"""The seeded generator: shapes, ranges, determinism, and the structure each configuration names."""
import numpy as np
import pytest

from paper_2510_00932_b200 import inputs


def test_workload_table_matches_the_named_configurations():
    w = inputs.WORKLOADS
    assert (w["c1"].n, w["c1"].dtype, w["c1"].seed, w["c1"].scalar) == (1 << 20, "f64", 0, 0.4)
    assert (w["c2"].n, w["c2"].dtype, w["c2"].seed, w["c2"].iterations) == (1 << 25, "f64", 1, 100)
    assert (w["c3"].n, w["c3"].dtype, w["c3"].seed, w["c3"].scalar) == (1 << 26, "f32", 2, 3.0)
    assert (w["c4"].n, w["c4"].dist, w["c4"].seed) == (1 << 28, "lognormal_signed", 3)
    assert (1 << 24) + 7 in inputs.SWEEP_SIZES and 2000896 in inputs.SWEEP_SIZES
    assert min(inputs.SWEEP_SIZES) == 1 << 16 and max(inputs.SWEEP_SIZES) == 1 << 29


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_arrays_are_seeded_and_in_range(name):
    w = inputs.WORKLOADS[name]
    n = 50_000
    a, b, c = inputs.make_arrays(w, n)
    a2, b2, c2 = inputs.make_arrays(w, n)
    for u, v in ((a, a2), (b, b2), (c, c2)):
        assert u.dtype == w.np_dtype and u.shape == (n,)
        assert inputs.checksum(u) == inputs.checksum(v)
    assert inputs.checksum(a) != inputs.checksum(b) != inputs.checksum(c)
    if w.dist == "uniform01":
        assert a.min() >= 0 and a.max() < 1
    elif w.dist == "uniform_pm1":
        assert a.min() >= -1 and a.max() < 1 and (a < 0).mean() > 0.4
    else:
        assert (a < 0).mean() > 0.4 and (a > 0).mean() > 0.4 and np.isfinite(a).all()
        logs = np.log(np.abs(a))
        assert abs(logs.mean()) < 0.1 and abs(logs.std() - 4.0) < 0.1


def test_special_values_cover_the_edge_classes():
    for t in ("f64", "f32"):
        v = inputs.special_values(t)
        assert np.isnan(v).sum() >= 3 and np.isinf(v).sum() == 2
        assert (v == 0).sum() == 2 and np.signbit(v[v == 0]).sum() == 1
        tiny = np.finfo(v.dtype).tiny
        assert ((np.abs(v) < tiny) & (v != 0)).sum() >= 2
