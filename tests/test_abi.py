"""The C-ABI library loads without a GPU and exports every symbol the header declares; host-side
status strings and tuning validation work. No kernel is launched here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def so():
    from paper_2510_00932_b200 import build, streamops
    build.build()
    return streamops


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "streamops.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(stream_[a-z0-9_]+|streamops_[a-z0-9_]+|shmem_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(so):
    names = _declared_symbols()
    assert len(names) >= 25 and "shmem_mix_u32" in names and "stream_triad_f64" in names and "streamops_chain_host_f32" in names
    L = so.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in include/streamops.h but not exported"


def test_status_strings_and_policy_names(so):
    assert so.status_string(0) == "ok"
    assert "overlap" in so.status_string(3)
    assert len({so.status_string(i) for i in range(8)}) == 8
    assert ".cs" in so.policy_name(2) and so.policy_name(99) == "unknown"


def test_tuning_table_validation_needs_no_gpu(so):
    so.reset_tuning()
    t = so.get_tuning("triad", "f64")
    assert t.vec_bytes in (16, 32) and t.threads in (128, 256, 512)
    so.set_tuning("triad", "f64", unroll=4, policy=3)
    assert so.get_tuning("triad", "f64").unroll == 4
    assert so.get_tuning("triad", "f32").unroll == t.unroll          # per (op, dtype)
    for bad in (dict(unroll=3), dict(vec_bytes=8), dict(threads=1024), dict(policy=9), dict(keep_mib=-1),
                dict(stages=1), dict(chunk_bytes=1000), dict(kind=2)):
        with pytest.raises(so.StreamopsError) as e:
            so.set_tuning("triad", "f64", **bad)
        assert e.value.status == 7
    so.reset_tuning()
    assert so.get_tuning("triad", "f64").unroll == t.unroll


def test_host_piece_size_validation(so):
    L = so.lib()
    assert L.streamops_set_host_piece_mib(0) == 7 and L.streamops_set_host_piece_mib(5000) == 7
    assert L.streamops_set_host_piece_mib(16) == 0


def test_binding_rejects_host_tensors(so):
    import torch
    x = torch.zeros(8, dtype=torch.float64)
    with pytest.raises(ValueError):
        so.copy(x, x.clone())
    with pytest.raises(TypeError):
        so._suffix(torch.zeros(2, dtype=torch.int32))


def test_product_path_has_no_oracle_dependency():
    pkg = os.path.join(ROOT, "paper_2510_00932_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f
