"""The CUDA-graph form of the five-kernel pass (host-overhead path at the paper's ARRAY_SIZE
values, Table 1): replays give bit-identical arrays and dot products to plain library calls, and
both match the oracle."""
import numpy as np
import pytest

from conftest import assert_bits_equal, bits
from paper_2510_00932_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("t,n", [("f64", 2000896), ("f32", 6000640), ("f64", 70_001)])
def test_graph_replay_matches_plain_calls_and_the_oracle(oracle, t, n):
    import torch
    from paper_2510_00932_b200 import hostpath, streamops as so
    so.reset_tuning()
    w = inputs.Workload("g", t, n, "uniform01", 4, 0.4, 1)
    a, b, c = inputs.make_arrays(w)
    ga, gb, gc = (torch.from_numpy(v.copy()).cuda() for v in (a, b, c))
    pa, pb, pc = (torch.from_numpy(v.copy()).cuda() for v in (a, b, c))
    pd = torch.zeros(1, dtype=pa.dtype, device="cuda")
    g = hostpath.ChainGraph(ga, gb, gc, w.scalar)        # its warm-up pass already advanced ga, gb, gc once
    so.chain(pa, pb, pc, pd, w.scalar)
    oa, ob, oc, od = oracle.chain(a, b, c, w.scalar)
    tol = 1e-12 if t == "f64" else 1e-5
    for it in range(4):
        g.replay()
        got = g.result()
        so.chain(pa, pb, pc, pd, w.scalar)
        torch.cuda.synchronize()
        oa, ob, oc, od = oracle.chain(oa, ob, oc, w.scalar)
        for name, x, y, o in (("a", ga, pa, oa), ("b", gb, pb, ob), ("c", gc, pc, oc)):
            assert (bits(x.cpu().numpy()) == bits(y.cpu().numpy())).all(), f"{name} iteration {it}"
            assert_bits_equal(x.cpu().numpy(), o, f"{name} vs oracle, iteration {it}")
        want = pd.item()
        assert np.array(got, dtype=a.dtype).view(bits(a).dtype) == np.array(want, dtype=a.dtype).view(bits(a).dtype)
        assert abs(got - od) <= tol * abs(od)
    so.check()


def test_protocol_timer_runs_and_reports_all_four(oracle):
    from paper_2510_00932_b200 import hostpath
    r = hostpath.time_protocols("f64", 2000896, 20, runs=2)
    assert set(r) == {"sync_each", "async_calls", "chain_call", "graph"}
    assert all(v["us_per_iter"] > 0 for v in r.values())
