"""Pins of the shared-memory exchange oracle against things other than itself: the closed form of
the round operator (trinomial coefficients from binomials, and an independent polynomial power,
both with Python integers), brute force on one tile written element by element, the algebra of the
operator (identity, composition, linearity, invertibility), and the fact that the output does not
degenerate at the paper's repetition counts (Table 1: 300 to 1500, default 600)."""
from math import comb

import numpy as np
import pytest

from paper_2510_00932_b200 import inputs

ROWS, COLS, TILE = 8, 1024, 8192
M32 = (1 << 32) - 1
PAPER_REPS = (300, 600, 900, 1200, 1500)


def trinomial_row_weights(rounds):
    """(1 + x + x^2)^R = sum_m T(R, m) x^m with T(R, m) = sum_i C(R, i) C(R - i, m - 2i) (i factors
    contribute x^2, m - 2i contribute x). With x the cyclic shift of the 8 rows, x^8 = 1, so row k
    of the result is sum_j w[j] * row (k + j) mod 8 with w[j] = sum over m = j mod 8 of T(R, m)."""
    w = [0] * ROWS
    for m in range(2 * rounds + 1):
        t = sum(comb(rounds, i) * comb(rounds - i, m - 2 * i) for i in range(max(0, m - rounds), m // 2 + 1))
        w[m % ROWS] += t
    return [v & M32 for v in w]


def polynomial_power_weights(rounds):
    """The same weights by square-and-multiply on coefficient lists modulo x^8 - 1 and 2^32."""
    def mul(a, b):
        c = [0] * ROWS
        for i, u in enumerate(a):
            for j, v in enumerate(b):
                c[(i + j) % ROWS] = (c[(i + j) % ROWS] + u * v) & M32
        return c
    result, base = [1] + [0] * (ROWS - 1), [1, 1, 1] + [0] * (ROWS - 3)
    while rounds:
        if rounds & 1:
            result = mul(result, base)
        base = mul(base, base)
        rounds >>= 1
    return result


def closed_form(x, rounds, weights=None):
    n = x.size
    out = np.empty(n, dtype=np.uint32)
    w = weights or polynomial_power_weights(rounds)
    tiles = n // TILE
    for t in range(tiles):
        tile = x[t * TILE:(t + 1) * TILE].reshape(ROWS, COLS).astype(object)
        for k in range(ROWS):
            acc = sum(w[j] * tile[(k + j) % ROWS] for j in range(ROWS))
            out[t * TILE + k * COLS:t * TILE + (k + 1) * COLS] = np.array([int(v) & M32 for v in acc], dtype=np.uint32)
    three = pow(3, rounds, 1 << 32)
    for i in range(tiles * TILE, n):
        out[i] = (int(x[i]) * three) & M32
    return out


def test_the_two_closed_forms_agree_with_each_other():
    for rounds in (0, 1, 2, 3, 7, 8, 9, 33, 133, 300, 600):
        assert trinomial_row_weights(rounds) == polynomial_power_weights(rounds)
    assert trinomial_row_weights(1) == [1, 1, 1, 0, 0, 0, 0, 0]
    assert trinomial_row_weights(2) == [1, 2, 3, 2, 1, 0, 0, 0]


@pytest.mark.parametrize("rounds", [0, 1, 2, 7, 8, 9, 31, 33, 133, 600, 1500])
def test_oracle_equals_the_closed_form(oracle, rounds):
    x = inputs.make_words(2 * TILE + 13, seed=11)
    weights = trinomial_row_weights(rounds) if rounds <= 600 else None
    assert (oracle.shmem_mix(x, rounds) == closed_form(x, rounds, weights)).all()


def test_one_tile_brute_force_element_by_element(oracle):
    x = inputs.make_words(TILE, seed=12)
    cur = [int(v) for v in x]
    for _ in range(3):
        nxt = [0] * TILE
        for i in range(TILE):
            k, c = divmod(i, COLS)
            nxt[i] = (cur[i] + cur[((k + 1) % ROWS) * COLS + c] + cur[((k + 2) % ROWS) * COLS + c]) & M32
        cur = nxt
    assert (oracle.shmem_mix(x, 3) == np.array(cur, dtype=np.uint32)).all()


def test_unit_impulse_spreads_upwards_with_trinomial_weights(oracle):
    # a single 1 in row 5: after R rounds row (5 - j) mod 8 holds the weight of x^j
    x = np.zeros(TILE, dtype=np.uint32)
    x[5 * COLS + 321] = 1
    R = 11
    got = oracle.shmem_mix(x, R).reshape(ROWS, COLS)
    w = trinomial_row_weights(R)
    for j in range(ROWS):
        assert int(got[(5 - j) % ROWS, 321]) == w[j]
    got[:, 321] = 0
    assert not got.any()                       # no other column is touched


def test_identity_composition_linearity_and_tail(oracle):
    x = inputs.make_words(3 * TILE + 100, seed=13)
    y = inputs.make_words(3 * TILE + 100, seed=14)
    assert (oracle.shmem_mix(x, 0) == x).all()
    assert (oracle.shmem_mix(oracle.shmem_mix(x, 5), 12) == oracle.shmem_mix(x, 17)).all()
    assert (oracle.shmem_mix(x + y, 9) == oracle.shmem_mix(x, 9) + oracle.shmem_mix(y, 9)).all()
    tail = oracle.shmem_mix(x, 3)[3 * TILE:]
    assert (tail == x[3 * TILE:] * np.uint32(27)).all()
    # a round takes rows k + 1 and k + 2, not k - 1 and k - 2, and takes each exactly once
    t = np.zeros(TILE, dtype=np.uint32); t[2 * COLS] = 7
    r = oracle.shmem_mix(t, 1).reshape(ROWS, COLS)
    assert [int(r[k, 0]) for k in range(ROWS)] == [7, 7, 7, 0, 0, 0, 0, 0]
    t = np.zeros(TILE, dtype=np.uint32); t[0] = 5             # row 0 reaches rows 7 and 6 around the cycle
    r = oracle.shmem_mix(t, 1).reshape(ROWS, COLS)
    assert [int(r[k, 0]) for k in range(ROWS)] == [5, 0, 0, 0, 0, 0, 5, 5]
    assert oracle.shmem_mix(np.zeros(0, dtype=np.uint32), 4).size == 0
    small = inputs.make_words(5, seed=15)
    assert (oracle.shmem_mix(small, 2) == small * np.uint32(9)).all()


@pytest.mark.parametrize("rounds", PAPER_REPS)
def test_output_is_not_degenerate(oracle, rounds):
    """At every repetition count of the paper the result still depends on the input and on the
    count: all eight row weights are non-zero, a non-zero input gives a non-zero output, one round
    fewer gives a different output, and changing one input word changes the output."""
    assert all(polynomial_power_weights(rounds))
    x = inputs.make_words(2 * TILE + 50, seed=17)
    out = oracle.shmem_mix(x, rounds)
    assert out[:2 * TILE].any() and out[2 * TILE:].any()
    fewer = oracle.shmem_mix(x, rounds - 1)
    assert (out != fewer).mean() > 0.99
    one = np.zeros(TILE + 3, dtype=np.uint32)
    one[3 * COLS + 9] = 1
    one[TILE + 1] = 1
    r = oracle.shmem_mix(one, rounds)
    assert all(int(v) != 0 for v in r[:TILE].reshape(ROWS, COLS)[:, 9])      # the impulse reaches every row
    assert int(r[TILE + 1]) == pow(3, rounds, 1 << 32) and r[TILE + 1] % 2 == 1


def test_a_round_can_be_undone(oracle):
    """The round is a bijection: (1 + x + x^2) has an inverse modulo x^8 - 1 and 2^32. Build the
    inverse's weights by Newton iteration with Python integers and apply them to the oracle's
    output: the input comes back, after 1 round and after 600."""
    def mul(a, b):
        c = [0] * ROWS
        for i, u in enumerate(a):
            for j, v in enumerate(b):
                c[(i + j) % ROWS] = (c[(i + j) % ROWS] + u * v) & M32
        return c
    f = [1, 1, 1] + [0] * (ROWS - 3)
    # modulo 2 the inverse is f^7 (the unit group of GF(2)[x]/(x+1)^8 has exponent 8); Newton lifts it
    g = f
    for _ in range(6):
        g = mul(g, f)
    for _ in range(6):                         # each step doubles the power of two the identity holds modulo
        fg = mul(f, g)
        two_minus = [(-v) & M32 for v in fg]
        two_minus[0] = (two_minus[0] + 2) & M32
        g = mul(g, two_minus)
    assert mul(f, g) == [1] + [0] * (ROWS - 1)
    x = inputs.make_words(TILE, seed=18)
    for rounds in (1, 600):
        inv = [1] + [0] * (ROWS - 1)
        base, e = g, rounds
        while e:
            if e & 1:
                inv = mul(inv, base)
            base = mul(base, base)
            e >>= 1
        back = closed_form(oracle.shmem_mix(x, rounds), 0, inv)
        assert (back == x).all()


def test_threaded_form_only_partitions(oracle):
    x = inputs.make_words(7 * TILE + 9, seed=16)
    for nt in (2, 3, 16):
        assert (oracle.shmem_mix(x, 20, nthreads=nt) == oracle.shmem_mix(x, 20)).all()
