"""Parity of the shared-memory exchange microkernel (shmem_mix_u32, through the C ABI) with the CPU
oracle: bit-exact on every word, at sizes spanning no tile, one tile, several grid-strides of tiles
and a ragged tail, at every access width, in place, and at the size the benchmark times."""
import os

import numpy as np
import pytest

from paper_2510_00932_b200 import inputs

pytestmark = pytest.mark.gpu
TILE = 8192
GUARD = 64
SENTINEL = 0xDEADBEEF


@pytest.fixture(scope="module")
def torch():
    import torch as _torch
    if not _torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return _torch


@pytest.fixture(scope="module")
def so(torch):
    from paper_2510_00932_b200 import streamops
    streamops.lib()
    yield streamops
    streamops.set_shmem_width(16)


def _guarded(torch, host, offset=0):
    raw = np.full(GUARD + offset + host.size + GUARD, SENTINEL, dtype=np.uint32)
    raw[GUARD + offset:GUARD + offset + host.size] = host
    full = torch.from_numpy(raw.view(np.int32)).cuda()
    return full, full[GUARD + offset:GUARD + offset + host.size]


def _check(torch, full, view, want, offset):
    got = view.cpu().numpy().view(np.uint32)
    assert (got == want).all(), f"{int((got != want).sum())} of {want.size} words differ, first at {int(np.flatnonzero(got != want)[0])}"
    f = full.cpu().numpy().view(np.uint32)
    assert (f[:GUARD + offset] == SENTINEL).all() and (f[GUARD + offset + want.size:] == SENTINEL).all(), "guard words overwritten"


@pytest.mark.parametrize("width", [4, 8, 16])
@pytest.mark.parametrize("n", [1, 5, TILE - 1, TILE, TILE + 1, 3 * TILE + 77, 40 * TILE + 1000])
def test_sizes_and_widths(so, torch, oracle, width, n):
    so.set_shmem_width(width)
    x = inputs.make_words(n, seed=21)
    for rounds in (0, 1, 7, 8, 33):
        fx, dx = _guarded(torch, x)
        fo, do = _guarded(torch, np.zeros(n, dtype=np.uint32))
        before = so.launch_count()
        so.shmem_mix(dx, do, rounds)
        torch.cuda.synchronize()
        assert so.launch_count() - before == 1
        _check(torch, fo, do, oracle.shmem_mix(x, rounds), 0)
        _check(torch, fx, dx, x, 0)                       # the input is left alone


@pytest.mark.parametrize("offset", [0, 1, 2, 3, 4])
def test_less_aligned_arrays_take_narrower_accesses_same_result(so, torch, oracle, offset):
    so.set_shmem_width(16)
    n = 5 * TILE + 123
    x = inputs.make_words(n, seed=22)
    fx, dx = _guarded(torch, x, offset)
    fo, do = _guarded(torch, np.zeros(n, dtype=np.uint32), offset)
    so.shmem_mix(dx, do, 19)
    torch.cuda.synchronize()
    _check(torch, fo, do, oracle.shmem_mix(x, 19), offset)


def test_in_place_and_more_tiles_than_blocks(so, torch, oracle):
    so.set_shmem_width(16)
    n = 2500 * TILE + 4097                                # more tiles than resident blocks: the tile loop wraps
    x = inputs.make_words(n, seed=23)
    fx, dx = _guarded(torch, x)
    so.shmem_mix(dx, dx, 5)
    torch.cuda.synchronize()
    _check(torch, fx, dx, oracle.shmem_mix(x, 5, nthreads=len(os.sched_getaffinity(0))), 0)


def test_tail_block_still_busy_with_its_last_tile(so, torch, oracle):
    # the block that owns the ragged tail also owns tiles; its warps reach the tail at different times
    so.set_shmem_width(16)
    for tiles, tail, rounds in ((2220 + 280, 8191, 64), (741, 4097, 200), (3, 5000, 300)):
        n = tiles * TILE + tail
        x = inputs.make_words(n, seed=24)
        want = oracle.shmem_mix(x, rounds, nthreads=len(os.sched_getaffinity(0)))
        dx = torch.from_numpy(x.view(np.int32)).cuda()
        do = torch.empty_like(dx)
        for _ in range(4):
            do.zero_()
            so.shmem_mix(dx, do, rounds)
            torch.cuda.synchronize()
            assert (do.cpu().numpy().view(np.uint32) == want).all()


@pytest.mark.parametrize("rounds", [600, 1500])
def test_benchmark_size_at_the_paper_default_and_largest_repetition_counts(so, torch, oracle, rounds):
    so.set_shmem_width(16)
    n = (1 << 24) + 4099                                  # the benchmark's tile count plus a ragged tail
    x = inputs.make_words(n, seed=5)
    dx = torch.from_numpy(x.view(np.int32)).cuda()
    do = torch.empty_like(dx)
    so.shmem_mix(dx, do, rounds)
    torch.cuda.synchronize()
    want = oracle.shmem_mix(x, rounds, nthreads=len(os.sched_getaffinity(0)))
    got = do.cpu().numpy().view(np.uint32)
    assert (got == want).all()
    # the comparison is not one of zeros with zeros, and a kernel that stopped a round early fails it
    assert inputs.checksum(want) != 0 and np.count_nonzero(want) > 0.99 * n
    fewer = oracle.shmem_mix(x[:3 * TILE], rounds - 1)
    assert (got[:3 * TILE] != fewer).mean() > 0.99


def test_argument_errors(so, torch):
    import ctypes
    L = so.lib()
    x = torch.zeros(3 * TILE, dtype=torch.int32, device="cuda")
    p = x.data_ptr()
    assert L.shmem_mix_u32(None, None, 3, 0, None) == 0                  # n == 0: nothing to do
    assert L.shmem_mix_u32(None, p, 3, 8, None) == 1
    assert L.shmem_mix_u32(p + 2, p + 4 * TILE, 3, 8, None) == 2
    assert L.shmem_mix_u32(p, p + 4, 3, TILE, None) == 3                 # partial overlap
    assert L.streamops_set_shmem_width(12) == 7
    with pytest.raises(ValueError):
        so.shmem_mix(x.float(), x.float(), 1)
