"""Random sequences of the four elementwise kernels (and Dot in between) over three arrays, with the
default automatic traversal direction: whatever direction each call picks from the call before it,
every array stays bit-identical to the same sequence run through the CPU oracle."""
import numpy as np
import pytest

from conftest import assert_bits_equal
from paper_2510_00932_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("t,n,seed", [("f64", (1 << 21) + 37, 41), ("f32", (1 << 22) + 5, 42), ("f64", 4097, 43)])
def test_random_call_sequences_match_the_oracle(oracle, t, n, seed):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00932_b200 import streamops as so
    so.lib(); so.reset_tuning()
    w = inputs.sweep_workload(t, n)
    host = list(inputs.make_arrays(w))
    dev = [torch.from_numpy(v.copy()).cuda() for v in host]
    dd = torch.zeros(1, dtype=dev[0].dtype, device="cuda")
    rng = np.random.Generator(np.random.PCG64(seed))
    tol = 1e-12 if t == "f64" else 1e-5
    for step in range(40):
        op = ("copy", "scale", "add", "triad", "dot")[int(rng.integers(0, 5))]
        i, j, k = (int(v) for v in rng.permutation(3))
        s = float(rng.choice([0.4, -1.25, 0.75]))
        if op == "copy":
            so.copy(dev[i], dev[k]); host[k] = oracle.copy(host[i])
        elif op == "scale":
            inplace = bool(rng.integers(0, 2))
            o = i if inplace else k
            so.scale(dev[i], dev[o], s); host[o] = oracle.scale(host[i], s)
        elif op == "add":
            o = (k, i, j)[int(rng.integers(0, 3))]                      # fresh output, or in place on x or on y
            so.add(dev[i], dev[j], dev[o]); host[o] = oracle.add(host[i], host[j])
        elif op == "triad":
            o = (k, i, j)[int(rng.integers(0, 3))]
            so.triad(dev[i], dev[j], dev[o], s); host[o] = oracle.triad(host[i], host[j], s)
        else:
            so.dot(dev[i], dev[j], dd)
            want = oracle.dot(host[i], host[j])
            assert abs(dd.item() - want) <= tol * max(abs(want), tol * oracle.dot_abs(host[i], host[j]))
        if step % 8 == 7 or step == 39:
            for a in range(3):
                assert_bits_equal(dev[a].cpu().numpy(), host[a], f"array {a} after step {step} ({op})")
    so.check()
