"""Pins of the shared-memory exchange oracle against things other than itself: the closed form of
the round operator (binomial coefficients, computed with Python integers), brute force on one tile
written element by element, and the algebra of the operator (identity, composition, linearity)."""
from math import comb

import numpy as np
import pytest

from paper_2510_00932_b200 import inputs

ROWS, COLS, TILE = 8, 1024, 8192
M32 = (1 << 32) - 1


def closed_form(x, rounds):
    """(I + P)^R = sum_j C(R, j) P^j with P the cyclic row shift: row k of the result is
    sum_j C(R, j) * row (k + j) mod 8; tail words are multiplied by 2^R. Python integers."""
    n = x.size
    out = np.empty(n, dtype=np.uint32)
    coef = [0] * ROWS
    for j in range(rounds + 1):
        coef[j % ROWS] += comb(rounds, j)
    coef = [c & M32 for c in coef]
    tiles = n // TILE
    for t in range(tiles):
        tile = x[t * TILE:(t + 1) * TILE].reshape(ROWS, COLS).astype(object)
        for k in range(ROWS):
            acc = sum(coef[j] * tile[(k + j) % ROWS] for j in range(ROWS))
            out[t * TILE + k * COLS:t * TILE + (k + 1) * COLS] = np.array([int(v) & M32 for v in acc], dtype=np.uint32)
    for i in range(tiles * TILE, n):
        out[i] = (int(x[i]) << rounds) & M32 if rounds < 64 else 0
    return out


@pytest.mark.parametrize("rounds", [0, 1, 2, 7, 8, 9, 31, 33, 600])
def test_oracle_equals_the_binomial_closed_form(oracle, rounds):
    x = inputs.make_words(2 * TILE + 13, seed=11)
    assert (oracle.shmem_mix(x, rounds) == closed_form(x, rounds)).all()


def test_one_tile_brute_force_element_by_element(oracle):
    x = inputs.make_words(TILE, seed=12)
    cur = [int(v) for v in x]
    for _ in range(3):
        nxt = [0] * TILE
        for i in range(TILE):
            k, c = divmod(i, COLS)
            nxt[i] = (cur[i] + cur[((k + 1) % ROWS) * COLS + c]) & M32
        cur = nxt
    assert (oracle.shmem_mix(x, 3) == np.array(cur, dtype=np.uint32)).all()


def test_unit_impulse_spreads_upwards_with_binomial_weights(oracle):
    # a single 1 in row 5: after R rounds row (5 - j) mod 8 holds sum of C(R, j') over j' = j mod 8
    x = np.zeros(TILE, dtype=np.uint32)
    x[5 * COLS + 321] = 1
    R = 11
    got = oracle.shmem_mix(x, R).reshape(ROWS, COLS)
    for j in range(ROWS):
        want = sum(comb(R, jj) for jj in range(j, R + 1, ROWS)) & M32
        assert int(got[(5 - j) % ROWS, 321]) == want
    got[:, 321] = 0
    assert not got.any()                       # no other column is touched


def test_identity_composition_linearity_and_tail(oracle):
    x = inputs.make_words(3 * TILE + 100, seed=13)
    y = inputs.make_words(3 * TILE + 100, seed=14)
    assert (oracle.shmem_mix(x, 0) == x).all()
    assert (oracle.shmem_mix(oracle.shmem_mix(x, 5), 12) == oracle.shmem_mix(x, 17)).all()
    assert (oracle.shmem_mix(x + y, 9) == oracle.shmem_mix(x, 9) + oracle.shmem_mix(y, 9)).all()
    tail = oracle.shmem_mix(x, 3)[3 * TILE:]
    assert (tail == x[3 * TILE:] * np.uint32(8)).all()
    assert not oracle.shmem_mix(x, 32)[3 * TILE:].any()         # 2^32 = 0 modulo 2^32
    # a round is not the opposite shift: row k must take row k + 1, not row k - 1
    t = np.zeros(TILE, dtype=np.uint32); t[2 * COLS] = 7
    r = oracle.shmem_mix(t, 1).reshape(ROWS, COLS)
    assert r[1, 0] == 7 and r[2, 0] == 7 and r[3, 0] == 0
    assert oracle.shmem_mix(np.zeros(0, dtype=np.uint32), 4).size == 0
    small = inputs.make_words(5, seed=15)
    assert (oracle.shmem_mix(small, 2) == small * np.uint32(4)).all()


def test_threaded_form_only_partitions(oracle):
    x = inputs.make_words(7 * TILE + 9, seed=16)
    for nt in (2, 3, 16):
        assert (oracle.shmem_mix(x, 20, nthreads=nt) == oracle.shmem_mix(x, 20)).all()
