"""stream_dot_noalloc_f64, the Dot for callers that cannot allocate device memory (their whole
device belongs to a memory pool already, or they may not take the allocator's lock where they
need the result). Its partial sums live in a fixed array inside the library, shared by every
call, so the interesting failure is a second call that trips over what the first one left
behind: the test makes two calls in a row, on different data, and checks each against the
regular stream_dot_f64 through the C ABI. Collected last on purpose (file name), so a run that
stops at the first failure has already run everything else. Works alone in a fresh process too:
it relies on no set-up done by other tests."""
import ctypes

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

REL_TOL = 1e-12          # the tolerance the fp64 Dot parity tests use


def _arrays(torch, n, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    x = (2.0 * rng.random(n) - 1.0) * np.exp2(rng.integers(-8, 8, size=n).astype(np.float64))
    y = (2.0 * rng.random(n) - 1.0) * np.exp2(rng.integers(-8, 8, size=n).astype(np.float64))
    return torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()


def test_no_alloc_dot_matches_the_regular_dot_on_two_calls_in_a_row():
    import torch
    assert torch.cuda.is_available()
    from paper_2510_00932_b200 import streamops as so
    L = so.lib()
    stream = torch.cuda.current_stream().cuda_stream
    out_na = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")
    out_ref = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")
    # first call: several spans and a ragged end; second call: a different length and data, so
    # stale partial sums or a ticket left mid-count from the first call would show
    for n, seed in (((1 << 20) + 12345, 1), (3 * 65536 + 7, 2), (5, 3)):
        x, y = _arrays(torch, n, seed)
        assert L.stream_dot_noalloc_f64(x.data_ptr(), y.data_ptr(), out_na.data_ptr(), 0.0, n, stream) == 0
        assert L.stream_dot_f64(x.data_ptr(), y.data_ptr(), out_ref.data_ptr(), 0.0, n, stream) == 0
        torch.cuda.synchronize()
        got, want = out_na.item(), out_ref.item()
        scale = float((x.abs() * y.abs()).sum().item())
        assert abs(got - want) <= REL_TOL * max(abs(want), 1e-3 * scale), (n, got, want)
        # repeated on the same data: identical bits (fixed summation order)
        again = torch.zeros(1, dtype=torch.float64, device="cuda")
        assert L.stream_dot_noalloc_f64(x.data_ptr(), y.data_ptr(), again.data_ptr(), 0.0, n, stream) == 0
        torch.cuda.synchronize()
        assert again.cpu().numpy().view(np.uint64)[0] == out_na.cpu().numpy().view(np.uint64)[0]
    # element-aligned but not 32-byte-aligned inputs take the scalar path with the same answer
    x, y = _arrays(torch, 200_001, 4)
    so.dot_noalloc(x[1:], y[1:], out_na)
    so.dot(x[1:], y[1:], out_ref)
    torch.cuda.synchronize()
    assert abs(out_na.item() - out_ref.item()) <= REL_TOL * abs(out_ref.item())


def test_no_alloc_dot_argument_checks():
    import torch
    from paper_2510_00932_b200 import streamops as so
    L = so.lib()
    x = torch.ones(1024, dtype=torch.float64, device="cuda")
    out = torch.full((1,), 7.0, dtype=torch.float64, device="cuda")
    p, o = x.data_ptr(), out.data_ptr()
    too_big = so.DOT_NOALLOC_MAX_N + 1
    # rejected before anything is launched or touched: the buffers are far smaller than n
    assert L.stream_dot_noalloc_f64(p, p, o, 0.0, ctypes.c_size_t(too_big), None) == 8
    assert "no-allocation" in so.status_string(8)
    assert L.stream_dot_noalloc_f64(None, p, o, 0.0, 8, None) == 1
    assert L.stream_dot_noalloc_f64(p + 4, p, o, 0.0, 8, None) == 2
    assert L.stream_dot_noalloc_f64(p, p, p + 8, 0.0, 8, None) == 3
    torch.cuda.synchronize()
    assert out.item() == 7.0
    assert L.stream_dot_noalloc_f64(p, p, o, 0.0, 0, None) == 0        # n = 0 writes +0
    torch.cuda.synchronize()
    assert out.item() == 0.0
    assert L.stream_dot_noalloc_f64(p, p, o, 0.0, 1024, None) == 0
    torch.cuda.synchronize()
    assert out.item() == 1024.0
