"""Pins for the oracle's Dot (Table 1, "Dot"): exact rational / big-integer dot products,
closed forms, unit vectors, cancellation patterns a plain sum gets wrong, and a second
summation route. CPU only."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import exact

ULP64 = 2.0**-52


def _rand(dtype, n, seed, spread=8):
    rng = np.random.Generator(np.random.PCG64(seed))
    mag = np.exp2(rng.integers(-spread, spread, size=n).astype(np.float64))
    return ((2.0 * rng.random(n) - 1.0) * mag).astype(dtype)


def _within_ulps(got: float, truth: Fraction, ulps: float, fmt="f64"):
    want = exact.round_to_format(truth, fmt)
    eps = ULP64 if fmt == "f64" else 2.0**-23
    return abs(Fraction(got) - truth) <= Fraction(ulps * eps) * abs(Fraction(want)) or got == want


@pytest.mark.parametrize("n", [0, 1, 2, 3, 7, 33, 64])
@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_dot_tiny_against_exact_rational(oracle, dtype, n):
    x, y = _rand(dtype, n, 100 + n), _rand(dtype, n, 200 + n)
    truth = exact.dot_exact_fraction(x, y)
    got = oracle.dot(x, y)
    assert _within_ulps(got, truth, 1.0), (got, float(truth))
    if n == 0:
        assert got == 0.0 and not np.signbit(got)


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_dot_large_against_exact_bigint(oracle, dtype):
    n = 100_003
    x, y = _rand(dtype, n, 1, spread=20), _rand(dtype, n, 2, spread=20)
    truth = exact.dot_exact_bigint(x, y)
    assert exact.dot_exact_bigint(x[:50], y[:50]) == exact.dot_exact_fraction(x[:50], y[:50])
    got = oracle.dot(x, y)
    assert _within_ulps(got, truth, 1.0), (got, float(truth))
    # the all-cores combination reaches the same accuracy for every split
    for nt in (1, 2, 5, 8):
        assert _within_ulps(oracle.run_mt("dot", x, y, 0.0, nt), truth, 1.0)


def test_dot_survives_cancellation_that_breaks_a_plain_sum(oracle):
    """x.y with huge terms that cancel: the exact answer is the small remainder."""
    M = 2.0**60
    reps = 2000
    x = np.tile(np.array([M, 1.0, -M, 3.0]), reps)
    y = np.tile(np.array([M, 1.0, M, 0.5]), reps)
    truth = Fraction(reps) * Fraction(5, 2)
    assert exact.dot_exact_bigint(x, y) == truth
    assert oracle.dot(x, y) == float(truth)
    assert oracle.dot_longdouble(x, y) == float(truth)
    # this input does tell a compensated sum from a plain one
    plain = 0.0
    for u, v in zip(x.tolist(), y.tolist()):
        plain += u * v
    assert plain != float(truth)
    # ill-conditioned random data: second half built to cancel the first
    a = _rand(np.float64, 20000, 3, spread=30)
    b = _rand(np.float64, 20000, 4, spread=30)
    x2 = np.concatenate([a, -a, _rand(np.float64, 50, 5, 2)])
    y2 = np.concatenate([b, b, _rand(np.float64, 50, 6, 2)])
    truth2 = exact.dot_exact_bigint(x2, y2)
    assert truth2 == exact.dot_exact_fraction(x2[-50:], y2[-50:])
    # the published bound of the compensated dot product: u|s| + gamma_n^2 * sum|x_i y_i|
    u = Fraction(1, 2**53)
    gamma = (x2.size * u) / (1 - x2.size * u)
    mags = sum(abs(Fraction(p) * Fraction(q)) for p, q in zip(x2.tolist(), y2.tolist()))
    err = abs(Fraction(oracle.dot(x2, y2)) - truth2)
    assert err <= u * abs(truth2) + gamma * gamma * mags
    assert mags / abs(truth2) > 10**20, "the case must be badly conditioned to mean anything"
    # the same construction at a condition number the bound still resolves to the last bit
    a = _rand(np.float64, 20000, 3, spread=6)
    b = _rand(np.float64, 20000, 4, spread=6)
    x3 = np.concatenate([a, -a, _rand(np.float64, 50, 5, 2)])
    y3 = np.concatenate([b, b, _rand(np.float64, 50, 6, 2)])
    assert _within_ulps(oracle.dot(x3, y3), exact.dot_exact_bigint(x3, y3), 1.0)


def test_dot_product_error_term_is_kept(oracle):
    """Products whose rounding errors add up: dropping the fma error term loses them."""
    n = 4096
    x = np.full(n, 1.0 + 2.0**-30)
    y = np.full(n, 1.0 + 2.0**-30)            # x*y = 1 + 2^-29 + 2^-60: the last term is lost
    x = np.concatenate([x, [-(n * (1.0 + 2.0**-29))]])
    y = np.concatenate([y, [1.0]])
    truth = Fraction(n) * Fraction(1, 2**60)
    assert exact.dot_exact_bigint(x, y) == truth
    assert oracle.dot(x, y) == float(truth)


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_dot_closed_forms(oracle, dtype):
    n = 12345
    # constants that are powers of two: n*a*b exactly
    assert oracle.dot(np.full(n, 0.5, dtype), np.full(n, 4.0, dtype)) == 2.0 * n
    assert oracle.dot(np.ones(n, dtype), np.ones(n, dtype)) == float(n)
    # general constants: n*a*b within a rounding
    a, b = dtype(0.1), dtype(0.7)
    truth = n * Fraction(float(a)) * Fraction(float(b))
    assert _within_ulps(oracle.dot(np.full(n, a, dtype), np.full(n, b, dtype)), truth, 1.0)
    # unit vectors pick out one element exactly, at every position
    x = _rand(dtype, 257, 7)
    for k in range(257):
        e = np.zeros(257, dtype); e[k] = 1
        assert oracle.dot(x, e) == float(x[k])
    # symmetry
    y = _rand(dtype, 257, 8)
    assert oracle.dot(x, y) == oracle.dot(y, x)
    # sign: dot(x, -y) = -dot(x, y)
    assert oracle.dot(x, -y) == -oracle.dot(x, y)


def test_dot_f32_products_are_formed_exactly(oracle):
    """float products need 48 bits: forming them in float first would lose the low half."""
    x = np.array([1.0 + 2.0**-12] * 1000 + [-1000.0], np.float32)
    y = np.array([1.0 + 2.0**-12] * 1000 + [1.0 + 2.0**-11], np.float32)
    truth = exact.dot_exact_fraction(x, y)      # 1000 * 2^-24
    assert truth == Fraction(1000, 2**24)
    assert oracle.dot(x, y) == float(truth)


def test_dot_f32_rounds_to_float_as_the_output_type_requires(oracle):
    n = (1 << 24) + 7                           # n ones: the double result is exact, float is not
    ones = np.ones(n, np.float32)
    d = oracle.dot(ones, ones)
    assert d == float(n)
    assert np.float32(d) == np.float32(16777224.0)


def test_dot_two_routes_agree_on_workload_like_data(oracle):
    from paper_2510_00932_b200 import inputs
    for dist in ("uniform01", "lognormal_signed"):
        rng = np.random.Generator(np.random.PCG64(9))
        x = inputs.draw(rng, 200_000, "f64", dist)
        y = inputs.draw(rng, 200_000, "f64", dist)
        d1, d2 = oracle.dot(x, y), oracle.dot_longdouble(x, y)
        assert abs(d1 - d2) <= 2 * ULP64 * abs(d1)
        assert _within_ulps(d1, exact.dot_exact_bigint(x, y), 1.0)


def test_dot_abs_is_the_sum_of_magnitudes(oracle):
    x, y = _rand(np.float64, 1000, 10), _rand(np.float64, 1000, 11)
    truth = sum(abs(Fraction(float(u)) * Fraction(float(v))) for u, v in zip(x, y))
    assert abs(Fraction(oracle.dot_abs(x, y)) - truth) <= Fraction(1e-15) * truth
    xf, yf = x.astype(np.float32), y.astype(np.float32)
    truthf = sum(abs(Fraction(float(u)) * Fraction(float(v))) for u, v in zip(xf, yf))
    assert abs(Fraction(oracle.dot_abs(xf, yf)) - truthf) <= Fraction(1e-15) * truthf


def test_fold_adds_left_to_right_with_one_rounding_per_step(oracle):
    """The fold of per-GPU partial sums is pinned by inputs on which every other order, and any
    wider accumulator, gives a different double."""
    from fractions import Fraction
    from oracle import exact
    f = lambda *v: oracle.fold(np.array(v, dtype=np.float64))
    assert f() == 0.0 and f(3.5) == 3.5
    assert f(1e16, 1.0, -1e16) == 0.0                   # right-to-left or exact summation gives 1
    assert f(-1e16, 1e16, 1.0) == 1.0
    assert f(2.0 ** 53, 1.0, 1.0) == 2.0 ** 53          # pairwise (1 + 1 first) gives 2^53 + 2
    assert f(1.0, 1.0, 2.0 ** 53) == 2.0 ** 53 + 2.0
    rng = np.random.Generator(np.random.PCG64(77))
    p = rng.standard_normal(64) * np.exp(rng.uniform(-30, 30, 64))
    acc = Fraction(0)
    for v in p:                                          # exact rational step, rounded to double every time
        acc = Fraction(exact.round_to_format(acc + Fraction(float(v)), "f64"))
    assert oracle.fold(p) == float(acc)
