"""CPU oracle for the five streaming kernels and the shared-memory exchange microkernel -- TEST
INFRASTRUCTURE, not part of the product.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this package.
It wraps ``streamops_oracle.c`` (plain scalar C loops following the textbook definitions of the
paper's Copy / Mul / Add / Triad / Dot kernels, Table 1) for numpy arrays. It imports nothing
from the CUDA package and the CUDA package imports nothing from here.

Every function takes and returns host numpy arrays; none touches a GPU.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SOURCES = ["streamops_oracle.c", "streamops_oracle_mt.c", "shmem_oracle.c"]
_LIB_PATH = os.path.join(_HERE, "liboracle.so")
# contraction off: a*b+c must stay two rounded operations; no value-changing optimisation
CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-pthread"]

OPS = ("copy", "scale", "add", "triad", "dot")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than a source."""
    srcs = [os.path.join(_HERE, s) for s in _SOURCES]
    if not force and os.path.exists(_LIB_PATH):
        if all(os.path.getmtime(_LIB_PATH) >= os.path.getmtime(s) for s in srcs):
            return _LIB_PATH
    tmp = _LIB_PATH + f".tmp{os.getpid()}"
    subprocess.run(["gcc", *CFLAGS, "-o", tmp, *srcs, "-lm"], check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        dp, sz, dbl = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_double
        for t in ("f64", "f32"):
            getattr(_lib, f"oracle_copy_{t}").argtypes = [dp, dp, sz]
            getattr(_lib, f"oracle_scale_{t}").argtypes = [dp, dp, dbl, sz]
            getattr(_lib, f"oracle_add_{t}").argtypes = [dp, dp, dp, sz]
            getattr(_lib, f"oracle_triad_{t}").argtypes = [dp, dp, dp, dbl, sz]
            getattr(_lib, f"oracle_dot_{t}").argtypes = [dp, dp, sz]
            getattr(_lib, f"oracle_dot_{t}").restype = dbl
            getattr(_lib, f"oracle_dot_abs_{t}").argtypes = [dp, dp, sz]
            getattr(_lib, f"oracle_dot_abs_{t}").restype = dbl
            for name in ("copy", "scale", "add", "triad"):
                getattr(_lib, f"oracle_{name}_{t}").restype = None
        _lib.oracle_dot_f64_longdouble.argtypes = [dp, dp, sz]
        _lib.oracle_dot_f64_longdouble.restype = dbl
        _lib.oracle_fold_f64.argtypes = [dp, sz]
        _lib.oracle_fold_f64.restype = dbl
        _lib.oracle_run_mt.argtypes = [ctypes.c_int, ctypes.c_int, dp, dp, dp, dbl, sz,
                                       ctypes.c_int, ctypes.POINTER(ctypes.c_double)]
        _lib.oracle_run_mt.restype = ctypes.c_int
        _lib.oracle_shmem_mix_u32.argtypes = [dp, dp, ctypes.c_uint, sz]
        _lib.oracle_shmem_mix_u32.restype = None
        _lib.oracle_shmem_mix_u32_mt.argtypes = [dp, dp, ctypes.c_uint, sz, ctypes.c_int]
        _lib.oracle_shmem_mix_u32_mt.restype = ctypes.c_int
    return _lib


def _suffix(x: np.ndarray) -> str:
    if x.dtype == np.float64:
        return "f64"
    if x.dtype == np.float32:
        return "f32"
    raise TypeError(f"oracle handles float32/float64 arrays, got {x.dtype}")


def _check(*arrs):
    t = _suffix(arrs[0])
    for a in arrs:
        if not (isinstance(a, np.ndarray) and a.ndim == 1 and a.flags.c_contiguous):
            raise ValueError("oracle arguments are contiguous 1-D numpy arrays")
        if _suffix(a) != t or a.shape != arrs[0].shape:
            raise ValueError("oracle arguments share one dtype and one length")
    return t


def _p(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def copy(x: np.ndarray) -> np.ndarray:
    """Copy: out[i] = x[i], bit for bit."""
    t = _check(x)
    out = np.empty_like(x)
    getattr(lib(), f"oracle_copy_{t}")(_p(x), _p(out), x.size)
    return out


def scale(x: np.ndarray, scalar: float) -> np.ndarray:
    """Mul: out[i] = RN(s * x[i]), s rounded once to the array's precision."""
    t = _check(x)
    out = np.empty_like(x)
    getattr(lib(), f"oracle_scale_{t}")(_p(x), _p(out), float(scalar), x.size)
    return out


def add(x: np.ndarray, y: np.ndarray) -> np.ndarray:
    """Add: out[i] = RN(x[i] + y[i])."""
    t = _check(x, y)
    out = np.empty_like(x)
    getattr(lib(), f"oracle_add_{t}")(_p(x), _p(y), _p(out), x.size)
    return out


def triad(x: np.ndarray, y: np.ndarray, scalar: float) -> np.ndarray:
    """Triad: out[i] = RN(x[i] + RN(s * y[i])), two roundings."""
    t = _check(x, y)
    out = np.empty_like(x)
    getattr(lib(), f"oracle_triad_{t}")(_p(x), _p(y), _p(out), float(scalar), x.size)
    return out


def dot(x: np.ndarray, y: np.ndarray) -> float:
    """Dot: compensated sum of x[i]*y[i], returned as a Python float (double) for both
    precisions; round it to float32 yourself to compare an fp32 result."""
    t = _check(x, y)
    return float(getattr(lib(), f"oracle_dot_{t}")(_p(x), _p(y), x.size))


def dot_longdouble(x: np.ndarray, y: np.ndarray) -> float:
    """fp64 Dot by the long-double route (cross-check of :func:`dot`)."""
    if _check(x, y) != "f64":
        raise TypeError("long-double cross-check is for float64 arrays")
    return float(lib().oracle_dot_f64_longdouble(_p(x), _p(y), x.size))


def dot_abs(x: np.ndarray, y: np.ndarray) -> float:
    """Sum of |x[i]*y[i]| (condition-number numerator)."""
    t = _check(x, y)
    return float(getattr(lib(), f"oracle_dot_abs_{t}")(_p(x), _p(y), x.size))


def fold(partials: np.ndarray) -> float:
    """Left-to-right double-precision sum of per-GPU partial dot products (rank order)."""
    if not (isinstance(partials, np.ndarray) and partials.dtype == np.float64 and partials.ndim == 1
            and partials.flags.c_contiguous):
        raise ValueError("fold takes a contiguous 1-D float64 array")
    return float(lib().oracle_fold_f64(_p(partials), partials.size))


def run_mt(op: str, x: np.ndarray, y, scalar: float, nthreads: int, out=None):
    """All-cores form: the index range cut into ``nthreads`` contiguous pieces, each piece run
    by the single-thread oracle. Returns the output array, or the dot product as a float."""
    arrs = [x] if y is None else [x, y]
    t = _check(*arrs)
    code = OPS.index(op)
    res = ctypes.c_double(0.0)
    if op != "dot" and out is None:
        out = np.empty_like(x)
    rc = lib().oracle_run_mt(code, 1 if t == "f64" else 0, _p(x),
                             _p(y) if y is not None else None,
                             _p(out) if out is not None else None,
                             float(scalar), x.size, int(nthreads), ctypes.byref(res))
    if rc != 0:
        raise RuntimeError("oracle_run_mt failed")
    return float(res.value) if op == "dot" else out


def chain(a: np.ndarray, b: np.ndarray, c: np.ndarray, scalar: float):
    """One pass of the five kernels over the three arrays in the textbook STREAM dataflow:
    c <- a; b <- s*c; c <- a+b; a <- b+s*c; dot(a, b). Returns (a, b, c, dot)."""
    c = copy(a)
    b = scale(c, scalar)
    c = add(a, b)
    a = triad(b, c, scalar)
    return a, b, c, dot(a, b)


SHMEM_ROWS, SHMEM_COLS = 8, 1024
SHMEM_TILE = SHMEM_ROWS * SHMEM_COLS


def shmem_mix(x: np.ndarray, rounds: int, nthreads: int = 1) -> np.ndarray:
    """Shared-memory exchange microkernel (the definition is in shmem_oracle.c): tiles of 8 rows
    x 1024 columns of 32-bit words; a round adds to every row the two rows below it (cyclically,
    modulo 2^32); words past the last whole tile triple every round. ``nthreads`` > 1 only deals whole
    tiles to threads."""
    if not (isinstance(x, np.ndarray) and x.dtype == np.uint32 and x.ndim == 1 and x.flags.c_contiguous):
        raise ValueError("shmem_mix takes a contiguous 1-D uint32 array")
    if rounds < 0 or rounds >= 2 ** 32:
        raise ValueError("rounds out of range")
    out = np.empty_like(x)
    if nthreads <= 1:
        lib().oracle_shmem_mix_u32(_p(x), _p(out), int(rounds), x.size)
    elif lib().oracle_shmem_mix_u32_mt(_p(x), _p(out), int(rounds), x.size, int(nthreads)) != 0:
        raise RuntimeError("oracle_shmem_mix_u32_mt failed")
    return out
