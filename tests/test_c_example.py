"""The C ABI used from plain C: examples/five_kernels.c compiles against include/streamops.h and links
against libstreamops.so with gcc (no GPU needed for that); on a GPU it runs the five kernels on
constant arrays and checks their closed-form results itself."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "paper_2510_00932_b200", "examples", "five_kernels.c")


def _cuda_home():
    for c in (os.environ.get("CUDA_HOME"), "/usr/local/cuda"):
        if c and os.path.exists(os.path.join(c, "include", "cuda_runtime.h")):
            return c
    pytest.skip("no CUDA toolkit headers")


def _build(tmp_path):
    from paper_2510_00932_b200 import build
    build.build()
    cuda = _cuda_home()
    pkg = os.path.join(ROOT, "paper_2510_00932_b200")
    exe = str(tmp_path / "five_kernels")
    cmd = ["gcc", "-O2", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"), SRC,
           "-L", pkg, "-lstreamops", "-L", os.path.join(cuda, "lib64"), "-lcudart", f"-Wl,-rpath,{pkg}",
           f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}", "-o", exe]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    return exe


def test_c_example_compiles_and_links_against_the_header_and_the_library(tmp_path):
    exe = _build(tmp_path)
    assert os.path.getsize(exe) > 0


@pytest.mark.gpu
def test_c_example_runs_and_checks_its_own_results(tmp_path):
    exe = _build(tmp_path)
    r = subprocess.run([exe, str((1 << 22) + 5)], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "ok: n = 4194309" in r.stdout and "dot = 2621443.125" in r.stdout
    assert all(name in r.stdout for name in ("copy", "scale", "add", "triad", "dot"))
