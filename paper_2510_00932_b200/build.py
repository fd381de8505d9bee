"""Builds libstreamops.so in-tree with nvcc for sm_100a (one translation unit per kernel family,
compiled in parallel, then linked). No GPU is needed to build."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(HERE, "libstreamops.so")
SOURCES = ["api.cu", "elementwise.cu", "ew_copy.cu", "ew_scale.cu", "ew_add.cu", "ew_triad.cu",
           "dot.cu", "dot_comp.cu", "bulk.cu", "dot_noalloc.cu", "shmem.cu"]
# -fmad=false is a second guard beside the explicit *_rn intrinsics; Dot asks for fma() by name.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-fmad=false", "-Xcompiler", "-fPIC"]


def _newest_input() -> float:
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(HERE, "..", "include", "streamops.h"))
    deps.append(os.path.abspath(__file__))
    return max(os.path.getmtime(d) for d in deps)


CHECKED_LIB_PATH = os.path.join(HERE, "libstreamops_checked.so")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Builds libstreamops.so, or with ``checked`` the debugging build libstreamops_checked.so, whose
    register-vector kernels check every global-memory index before using it (-DSTREAMOPS_CHECK_INDICES)."""
    lib_path = CHECKED_LIB_PATH if checked else LIB_PATH
    obj_dir = OBJ_DIR + ("_checked" if checked else "")
    if not force and os.path.exists(lib_path) and os.path.getmtime(lib_path) >= _newest_input():
        return lib_path
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(obj_dir, exist_ok=True)
    extra = ["-DSTREAMOPS_CHECK_INDICES"] if checked else []

    def compile_one(src: str) -> str:
        obj = os.path.join(obj_dir, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *extra, *(["-Xptxas", "-v"] if verbose else []), "-c",
               os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(SOURCES))) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    tmp = lib_path + f".tmp{os.getpid()}"
    r = subprocess.run([nvcc, "-shared", "-o", tmp, *objs, "-cudart", "shared"], capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
