"""Pins for the oracle's elementwise kernels (Copy, Mul/scale, Add, Triad of the paper's Table 1).

The oracle is checked against things other than itself: exact rational arithmetic rounded once by
integer arithmetic, algebraic identities of IEEE-754 arithmetic, and crafted operands on which a
fused multiply-add, a swapped operand, a dropped term or a wrong scalar rounding gives different
bits. CPU only.
"""
from fractions import Fraction

import numpy as np
import pytest

from conftest import assert_bits_equal, bits
from oracle import exact
from paper_2510_00932_b200 import inputs

DTYPES = [np.float64, np.float32]


def _rand(dtype, n, seed, lo=-4.0, hi=4.0):
    rng = np.random.Generator(np.random.PCG64(seed))
    # mixed magnitudes so that rounding actually happens in sums and products
    mag = np.exp2(rng.integers(-12, 12, size=n).astype(np.float64))
    return ((lo + (hi - lo) * rng.random(n)) * mag).astype(dtype)


# ---------------------------------------------------------------- round_to_format itself
def test_rounding_helper_against_known_values():
    # ties to even at the 53-bit boundary, and float32 rounding of 0.4 and 0.1
    assert exact.round_to_format(Fraction(2**53 + 1), "f64") == float(2**53)
    assert exact.round_to_format(Fraction(2**53 + 3), "f64") == float(2**53 + 4)
    assert exact.round_to_format(Fraction(4, 10), "f32") == float(np.float32(0.4))
    assert exact.round_to_format(Fraction(1, 10), "f64") == 0.1
    # gradual underflow: half the smallest subnormal is a tie and rounds to even (zero)
    assert exact.round_to_format(Fraction(1, 2**1075), "f64") == 0.0
    assert exact.round_to_format(Fraction(3, 2**1075), "f64") == 2 * 5e-324
    assert exact.round_to_format(Fraction(2)**128, "f32") == float("inf")
    assert exact.round_to_format(-Fraction(2)**-149, "f32") == -float(np.float32(1e-45))


# ---------------------------------------------------------------- copy
@pytest.mark.parametrize("dtype", DTYPES)
def test_copy_is_identity_on_bit_patterns(oracle, dtype):
    t = "f64" if dtype == np.float64 else "f32"
    sp = inputs.special_values(t)
    # signalling NaNs must survive too: copy moves bits, it does not compute
    snan = (np.array([0x7FF0000000000001, 0xFFF4000000000000], dtype=np.uint64).view(np.float64)
            if t == "f64" else np.array([0x7F800001, 0xFFA00000], dtype=np.uint32).view(np.float32))
    x = np.concatenate([sp, snan, _rand(dtype, 1000, 1)])
    out = oracle.copy(x)
    assert out is not x and (bits(out) == bits(x)).all()
    assert oracle.copy(x[:0]).size == 0


# ---------------------------------------------------------------- scale
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("scalar", [0.4, 3.0, -0.3, 1e-3, 1.0 / 3.0])
def test_scale_equals_exact_product_rounded_once(oracle, dtype, scalar):
    x = _rand(dtype, 400, 2)
    assert_bits_equal(oracle.scale(x, scalar), exact.scale_exact(x, scalar), "scale vs exact")


@pytest.mark.parametrize("dtype", DTYPES)
def test_scale_identities(oracle, dtype):
    t = "f64" if dtype == np.float64 else "f32"
    x = np.concatenate([_rand(dtype, 500, 3), inputs.special_values(t)])
    finite = np.isfinite(x)
    # s = 1 is the identity; s = -1 flips the sign bit only
    assert_bits_equal(oracle.scale(x, 1.0), x, "scale by 1")
    signbit = np.uint64(1 << 63) if t == "f64" else np.uint32(1 << 31)
    flipped = (bits(x) ^ signbit).view(dtype)
    assert_bits_equal(oracle.scale(x, -1.0), flipped, "scale by -1")
    # s = 0 gives a zero whose sign is the product of the signs (finite operands)
    z = oracle.scale(x, 0.0)[finite]
    assert (z == 0).all() and (np.signbit(z) == np.signbit(x[finite])).all()
    zneg = oracle.scale(x, -0.0)[finite]
    assert (np.signbit(zneg) != np.signbit(x[finite])).all()
    # powers of two shift the exponent exactly (integers stay integers)
    ints = np.arange(-300, 300).astype(dtype)
    assert (oracle.scale(ints, 8.0) == ints * 8).all()
    assert (oracle.scale(ints * 8, 0.125) == ints).all()
    # constants
    c = np.full(77, 0.1, dtype=dtype)
    want = exact.round_to_format(exact.scalar_in_format(0.4, t) * Fraction(float(dtype(0.1))), t)
    assert (oracle.scale(c, 0.4) == dtype(want)).all()


def test_scale_f32_rounds_the_scalar_once_to_float(oracle):
    # multiplying in double and rounding the product would differ from multiplying by float(0.4)
    x = _rand(np.float32, 4000, 4)
    got = oracle.scale(x, 0.4)
    via_double = (x.astype(np.float64) * 0.4).astype(np.float32)
    assert (bits(got) != bits(via_double)).any(), "operands chosen must tell the two readings apart"
    assert_bits_equal(got[:300], exact.scale_exact(x[:300], 0.4), "scale f32 vs exact")


# ---------------------------------------------------------------- add
@pytest.mark.parametrize("dtype", DTYPES)
def test_add_equals_exact_sum_rounded_once(oracle, dtype):
    x, y = _rand(dtype, 400, 5), _rand(dtype, 400, 6)
    assert_bits_equal(oracle.add(x, y), exact.add_exact(x, y), "add vs exact")


@pytest.mark.parametrize("dtype", DTYPES)
def test_add_identities(oracle, dtype):
    x, y = _rand(dtype, 1000, 7), _rand(dtype, 1000, 8)
    assert_bits_equal(oracle.add(x, y), oracle.add(y, x), "add commutes")
    zero = np.zeros_like(x)
    assert_bits_equal(oracle.add(x, zero), x, "x + 0")
    # operands tell x + y apart from x - y and from x alone
    assert (bits(oracle.add(x, y)) != bits(x)).any()
    ints = np.arange(1000).astype(dtype)
    assert (oracle.add(ints, ints[::-1].copy()) == 999).all()
    # -0 + -0 = -0, +0 + -0 = +0 under round-to-nearest
    nz = np.array([-0.0, 0.0], dtype=dtype)
    out = oracle.add(nz, np.array([-0.0, -0.0], dtype=dtype))
    assert np.signbit(out[0]) and not np.signbit(out[1])


# ---------------------------------------------------------------- triad
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("scalar", [0.4, 3.0, -1.7])
def test_triad_equals_two_exact_roundings(oracle, dtype, scalar):
    x, y = _rand(dtype, 400, 9), _rand(dtype, 400, 10)
    assert_bits_equal(oracle.triad(x, y, scalar), exact.triad_exact(x, y, scalar), "triad vs exact")


@pytest.mark.parametrize("dtype", DTYPES)
def test_triad_is_add_after_scale_bitwise(oracle, dtype):
    t = "f64" if dtype == np.float64 else "f32"
    x = np.concatenate([_rand(dtype, 5000, 11), inputs.special_values(t)])
    y = np.concatenate([_rand(dtype, 5000, 12), inputs.special_values(t)[::-1]])
    for s in (0.4, 3.0):
        assert_bits_equal(oracle.triad(x, y, s), oracle.add(x, oracle.scale(y, s)), "triad = add o scale")


@pytest.mark.parametrize("dtype", DTYPES)
def test_triad_is_not_a_fused_multiply_add(oracle, dtype):
    """Operands on which one rounding (FMA) and two roundings differ: the oracle takes two."""
    x, y = _rand(dtype, 3000, 13), _rand(dtype, 3000, 14)
    two = exact.triad_exact(x[:600], y[:600], 0.4)
    one = exact.fma_exact(x[:600], y[:600], 0.4)
    differ = bits(two) != bits(one)
    assert differ.sum() >= 20, "sample must contain cases that tell FMA from mul+add"
    got = oracle.triad(x[:600], y[:600], 0.4)
    assert_bits_equal(got, two, "triad takes two roundings")
    assert (bits(got)[differ] != bits(one)[differ]).all()
    # a crafted triple: s*y = 1 + 2^-p (a tie after the first rounding), x = -1
    if dtype == np.float64:
        s, yv, xv = 1.0 + 2.0**-30, np.array([1.0 + 2.0**-30]), np.array([-1.0])
    else:
        s, yv, xv = 1.0 + 2.0**-13, np.array([1.0 + 2.0**-13], np.float32), np.array([-1.0], np.float32)
    assert_bits_equal(oracle.triad(xv, yv, s), exact.triad_exact(xv, yv, s), "crafted")
    assert bits(exact.triad_exact(xv, yv, s))[0] != bits(exact.fma_exact(xv, yv, s))[0]


@pytest.mark.parametrize("dtype", DTYPES)
def test_triad_operand_roles(oracle, dtype):
    """out = x + s*y: the scalar multiplies the SECOND operand (swapping them changes bits)."""
    x, y = _rand(dtype, 500, 15), _rand(dtype, 500, 16)
    got = oracle.triad(x, y, 3.0)
    assert_bits_equal(got, exact.triad_exact(x, y, 3.0), "x + s*y")
    assert (bits(got) != bits(exact.triad_exact(y, x, 3.0))).any()


# ---------------------------------------------------------------- the whole chain
@pytest.mark.parametrize("dtype,scalar", [(np.float64, 0.4), (np.float32, 3.0), (np.float32, 0.4)])
def test_chain_on_constants_follows_the_scalar_recurrence(oracle, dtype, scalar):
    """One pass c<-a; b<-s*c; c<-a+b; a<-b+s*c over constant arrays equals the same recurrence on
    three scalars evaluated exactly with one rounding per operation."""
    t = "f64" if dtype == np.float64 else "f32"
    n = 1000
    a0, b0, c0 = dtype(0.1), dtype(0.2), dtype(0.0)
    a = np.full(n, a0, dtype=dtype); b = np.full(n, b0, dtype=dtype); c = np.full(n, c0, dtype=dtype)
    s = exact.scalar_in_format(scalar, t)
    fa, fb, fc = Fraction(float(a0)), Fraction(float(b0)), Fraction(float(c0))
    rn = lambda q: Fraction(exact.round_to_format(q, t))
    for _ in range(3):
        a, b, c, d = oracle.chain(a, b, c, scalar)
        fc = fa
        fb = rn(s * fc)
        fc = rn(fa + fb)
        fa = rn(fb + rn(s * fc))
        assert (a == dtype(float(fa))).all() and (b == dtype(float(fb))).all() and (c == dtype(float(fc))).all()
        exact_dot = n * fa * fb
        tol = 1e-12 if t == "f64" else 1e-5
        assert abs(Fraction(d) - exact_dot) <= Fraction(tol) * abs(exact_dot)


@pytest.mark.parametrize("dtype", DTYPES)
def test_all_cores_form_matches_single_thread(oracle, dtype):
    x, y = _rand(dtype, 10007, 17), _rand(dtype, 10007, 18)
    for nt in (1, 2, 3, 8):
        assert_bits_equal(oracle.run_mt("copy", x, None, 0.0, nt), oracle.copy(x), "mt copy")
        assert_bits_equal(oracle.run_mt("scale", x, None, 0.4, nt), oracle.scale(x, 0.4), "mt scale")
        assert_bits_equal(oracle.run_mt("add", x, y, 0.0, nt), oracle.add(x, y), "mt add")
        assert_bits_equal(oracle.run_mt("triad", x, y, 0.4, nt), oracle.triad(x, y, 0.4), "mt triad")


def test_pins_catch_an_oracle_built_with_contraction(tmp_path):
    """Plant the classic mistake in the oracle itself: build it with FMA contraction allowed.
    The exact-arithmetic Triad pin must then fail, which shows the pin has teeth."""
    import ctypes, os, subprocess
    import oracle as orc
    if "fma" not in open("/proc/cpuinfo").read():
        pytest.skip("host CPU has no FMA instruction to contract into")
    src = os.path.join(os.path.dirname(orc.__file__), "streamops_oracle.c")
    so = str(tmp_path / "mutant.so")
    subprocess.run(["gcc", "-O2", "-std=gnu11", "-mfma", "-ffp-contract=fast", "-fPIC", "-shared",
                    "-o", so, src, "-lm"], check=True)
    mutant = ctypes.CDLL(so)
    x, y = _rand(np.float64, 600, 13), _rand(np.float64, 600, 14)
    out = np.empty_like(x)
    mutant.oracle_triad_f64(ctypes.c_void_p(x.ctypes.data), ctypes.c_void_p(y.ctypes.data),
                            ctypes.c_void_p(out.ctypes.data), ctypes.c_double(0.4), ctypes.c_size_t(x.size))
    assert (bits(out) != bits(exact.triad_exact(x, y, 0.4))).any()
    assert_bits_equal(out, exact.fma_exact(x, y, 0.4), "the mutant is the fused form")
