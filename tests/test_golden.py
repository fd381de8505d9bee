"""Stored oracle results (tests/golden/checksums.json, written by tests/golden/make_golden.py from
the oracle alone): on CPU the oracle and the seeded generator must still reproduce them; on a GPU
the CUDA path must produce arrays with the same word checksums and a dot product within tolerance."""
import importlib.util
import json
import os

import numpy as np
import pytest

from paper_2510_00932_b200 import inputs

HERE = os.path.dirname(os.path.abspath(__file__))
GOLDEN = json.load(open(os.path.join(HERE, "golden", "checksums.json")))


def test_oracle_and_generator_still_reproduce_the_stored_values(oracle):
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    now = mod.compute()
    assert now["chain"] == GOLDEN["chain"] and now["shmem_mix"] == GOLDEN["shmem_mix"]


@pytest.mark.gpu
@pytest.mark.parametrize("name", sorted(GOLDEN["chain"]))
def test_cuda_chain_matches_the_stored_checksums(name):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00932_b200 import streamops as so
    so.lib(); so.reset_tuning()
    g = GOLDEN["chain"][name]
    w = inputs.WORKLOADS[name]
    a, b, c = inputs.make_arrays(w, g["n"])
    assert [inputs.checksum(v) for v in (a, b, c)] == g["inputs"]
    da, db, dc = (torch.from_numpy(v).cuda() for v in (a, b, c))
    dd = torch.zeros(1, dtype=da.dtype, device="cuda")
    so.chain(da, db, dc, dd, w.scalar)
    torch.cuda.synchronize()
    assert [inputs.checksum(t.cpu().numpy()) for t in (da, db, dc)] == g["after_one_pass"]
    want = float.fromhex(g["dot"])
    assert abs(dd.item() - want) <= (1e-12 if w.dtype == "f64" else 1e-5) * abs(want)


@pytest.mark.gpu
@pytest.mark.parametrize("key", sorted(GOLDEN["shmem_mix"]))
def test_cuda_shmem_mix_matches_the_stored_checksums(key):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00932_b200 import streamops as so
    n, rounds = (int(v) for v in key.split("x"))
    x = inputs.make_words(n)
    assert inputs.checksum(x) == GOLDEN["shmem_mix"][key]["input"]
    dx = torch.from_numpy(x.view(np.int32)).cuda()
    do = torch.empty_like(dx)
    so.shmem_mix(dx, do, rounds)
    torch.cuda.synchronize()
    assert inputs.checksum(do.cpu().numpy().view(np.uint32)) == GOLDEN["shmem_mix"][key]["output"]
