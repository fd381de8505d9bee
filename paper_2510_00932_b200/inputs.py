"""Seeded synthetic inputs for the five streaming kernels (Copy, Mul/scale, Add, Triad, Dot).

The paper (Table 1, Section 5.2) runs these kernels on three arrays of ARRAY_SIZE elements and
does not publish the array contents, so the arrays here are synthetic stand-ins for those runs.
This module only draws random numbers and shapes them; it contains none of the arithmetic of the
five operations, and it is the one module that both the CUDA path's tests and the CPU oracle's
tests feed from.

Every workload is three host arrays a, b, c of one dtype, drawn in that order from
``numpy.random.Generator(numpy.random.PCG64(seed))``, plus the scalar ``s``.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One named configuration: dtype, length, distribution, seed and scalar."""

    name: str
    dtype: str          # "f64" | "f32"
    n: int
    dist: str           # "uniform01" | "uniform_pm1" | "lognormal_signed"
    seed: int
    scalar: float
    iterations: int     # timed iterations the configuration asks for

    @property
    def np_dtype(self):
        return np.float64 if self.dtype == "f64" else np.float32

    @property
    def itemsize(self) -> int:
        return 8 if self.dtype == "f64" else 4


# The named configurations. "c2" is the headline bandwidth workload.
WORKLOADS = {
    "c1": Workload("c1", "f64", 1 << 20, "uniform01", 0, 0.4, 10),
    "c2": Workload("c2", "f64", 1 << 25, "uniform01", 1, 0.4, 100),
    "c3": Workload("c3", "f32", 1 << 26, "uniform_pm1", 2, 3.0, 100),
    "c4": Workload("c4", "f64", 1 << 28, "lognormal_signed", 3, 0.4, 20),
}

# Size sweep (configuration 5): powers of two across the L2-to-HBM transition, one ragged size
# that exercises the tail path, and the three ARRAY_SIZE values of the paper's Table 1.
SWEEP_SIZES = [1 << k for k in range(16, 30)] + [(1 << 24) + 7, 2000896, 4000768, 6000640]
SWEEP_SEED = 4
SWEEP_SCALAR = 0.4


def sweep_workload(dtype: str, n: int) -> Workload:
    return Workload(f"c5_{dtype}_{n}", dtype, int(n), "uniform01", SWEEP_SEED, SWEEP_SCALAR, 20)


def draw(rng: np.random.Generator, n: int, dtype: str, dist: str) -> np.ndarray:
    """Draw one array of ``n`` values of the named distribution from ``rng``."""
    npdt = np.float64 if dtype == "f64" else np.float32
    if dist == "uniform01":
        return rng.random(n, dtype=npdt)
    if dist == "uniform_pm1":
        # 2u - 1 is exact in the array's own precision for u in [0, 1)
        u = rng.random(n, dtype=npdt)
        u *= npdt(2)
        u -= npdt(1)
        return u
    if dist == "lognormal_signed":
        # log-normal magnitudes (mu = 0, sigma = 4) with independent random signs
        g = rng.standard_normal(n)
        g *= 4.0
        np.exp(g, out=g)
        sign = rng.integers(0, 2, size=n, dtype=np.int8)
        g[sign == 0] *= -1.0
        return g.astype(npdt, copy=False)
    raise ValueError(f"unknown distribution {dist!r}")


def make_arrays(w: Workload, n: int | None = None):
    """Return the host arrays (a, b, c) of workload ``w``; ``n`` overrides the length
    (a prefix-independent redraw, used for bounded samples)."""
    n = w.n if n is None else int(n)
    rng = np.random.Generator(np.random.PCG64(w.seed))
    a = draw(rng, n, w.dtype, w.dist)
    b = draw(rng, n, w.dtype, w.dist)
    c = draw(rng, n, w.dtype, w.dist)
    return a, b, c


def checksum(arr: np.ndarray) -> int:
    """Sum of the array's raw words modulo 2**64: detects a numpy whose generator stream differs."""
    words = arr.view(np.uint64 if arr.dtype.itemsize == 8 else np.uint32)
    return int(np.add.reduce(words, dtype=np.uint64))


def special_values(dtype: str) -> np.ndarray:
    """Edge-case operands: signed zeros, subnormals, extremes, infinities and NaNs with payloads."""
    if dtype == "f64":
        bits = np.array([
            0x0000000000000000, 0x8000000000000000, 0x0000000000000001, 0x800FFFFFFFFFFFFF,
            0x0010000000000000, 0x7FEFFFFFFFFFFFFF, 0xFFEFFFFFFFFFFFFF, 0x7FF0000000000000,
            0xFFF0000000000000, 0x7FF8000000000000, 0x7FF8000000ABCDEF, 0xFFF80000DEADBEEF,
            0x3FF0000000000000, 0xBFF0000000000000, 0x3FD999999999999A, 0x4330000000000001,
        ], dtype=np.uint64)
        return bits.view(np.float64)
    bits = np.array([
        0x00000000, 0x80000000, 0x00000001, 0x807FFFFF, 0x00800000, 0x7F7FFFFF, 0xFF7FFFFF,
        0x7F800000, 0xFF800000, 0x7FC00000, 0x7FC0ABCD, 0xFFC0BEEF, 0x3F800000, 0xBF800000,
        0x3ECCCCCD, 0x4B000001,
    ], dtype=np.uint32)
    return bits.view(np.float32)


def make_words(n: int, seed: int = 5) -> np.ndarray:
    """Uniform random 32-bit words for the shared-memory exchange microkernel (PCG64 stream)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, 1 << 32, size=int(n), dtype=np.uint32)


def make_cancelling(n: int, dtype: str = "f64", seed: int = 6, log2_big: int = 40):
    """Two arrays whose dot product cancels heavily: shuffled triples x = (A, r, -A), y = (B, s, B)
    with |A*B| about 2**log2_big times |r*s|, so that the large products cancel in pairs and only
    the sum of the r*s survives (condition number about 2**(log2_big + 1)). Values are random, no
    arithmetic of the kernels under test is involved. n is rounded down to a multiple of 3."""
    rng = np.random.Generator(np.random.PCG64(seed))
    t = n // 3
    np_t = np.float64 if dtype == "f64" else np.float32
    half = log2_big // 2
    A = (rng.uniform(1.0, 2.0, t) * 2.0 ** half).astype(np_t)
    B = (rng.uniform(1.0, 2.0, t) * 2.0 ** (log2_big - half)).astype(np_t)
    r = rng.uniform(-1.0, 1.0, t).astype(np_t)
    s = rng.uniform(-1.0, 1.0, t).astype(np_t)
    x = np.concatenate([A, r, -A])
    y = np.concatenate([B, s, B])
    perm = rng.permutation(3 * t)
    return np.ascontiguousarray(x[perm]), np.ascontiguousarray(y[perm])
