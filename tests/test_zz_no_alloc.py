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


SPAN = 65536             # elements per partial sum of the fixed scratch


@pytest.mark.parametrize("n", [1, SPAN - 1, SPAN, SPAN + 1, 3 * SPAN + 7, 1 << 28])
def test_no_alloc_dot_against_the_cpu_oracle_at_span_boundaries_and_the_largest_n(oracle, n):
    """Against the compensated CPU oracle, not against the library's other Dot: lengths that end
    just before, on and just after the boundary between two partial sums, several spans plus a
    ragged end, and the largest n the fixed scratch covers (all 4,096 partial sums in use)."""
    import os
    import torch
    from paper_2510_00932_b200 import streamops as so
    rng = np.random.Generator(np.random.PCG64(40 + n % 1000))
    x, y = rng.random(n) - 0.25, rng.random(n) - 0.25
    want = oracle.run_mt("dot", x, y, 0.0, len(os.sched_getaffinity(0))) if n > (1 << 24) else oracle.dot(x, y)
    dx, dy = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    out = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")
    so.dot_noalloc(dx, dy, out)
    torch.cuda.synchronize()
    assert abs(out.item() - want) <= REL_TOL * abs(want), (n, out.item(), want)
    if n > 8:                                           # element-aligned, not vector-aligned: the scalar path
        w1 = oracle.dot(x[1:], y[1:]) if n <= (1 << 24) else None
        if w1 is not None:
            so.dot_noalloc(dx[1:], dy[1:], out)
            torch.cuda.synchronize()
            assert abs(out.item() - w1) <= REL_TOL * abs(w1)


def test_no_alloc_dot_with_a_unit_vector_returns_that_element_exactly():
    """dot(x, e_k) = x[k] exactly for k at the first and last element of a span, of a tile inside
    a span and of the ragged end: every index is visited once, none twice, none skipped."""
    import torch
    from paper_2510_00932_b200 import streamops as so
    n = 5 * SPAN + 1234
    rng = np.random.Generator(np.random.PCG64(77))
    x = rng.standard_normal(n)
    dx = torch.from_numpy(x).cuda()
    e = torch.zeros(n, dtype=torch.float64, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    ks = [0, 1, 3, 4, 8191, 8192, SPAN - 1, SPAN, SPAN + 1, 2 * SPAN - 1, 2 * SPAN, 5 * SPAN - 1, 5 * SPAN,
          5 * SPAN + 1231, 5 * SPAN + 1232, n - 1]
    for k in ks:
        e[k] = 1.0
        so.dot_noalloc(dx, e, out)
        torch.cuda.synchronize()
        assert out.item() == x[k], k
        e[k] = 0.0


def test_no_alloc_dot_leaves_free_device_memory_alone_and_counts_its_launch():
    """After one warm call (which makes the CUDA runtime load the kernel's module), further calls --
    on more data than before -- must not change the amount of free device memory, and each adds
    one to the library's launch count. Run in a fresh process, so that the regular Dot's workspace
    does not exist yet: creating it afterwards lowers free memory, which shows that the
    no-allocation calls had not created it."""
    import subprocess
    import sys
    code = r"""
import torch, sys
from paper_2510_00932_b200 import streamops as so
L = so.lib()
x = torch.ones(1 << 22, dtype=torch.float64, device="cuda")
out = torch.zeros(1, dtype=torch.float64, device="cuda")
s = torch.cuda.current_stream().cuda_stream
assert L.stream_dot_noalloc_f64(x.data_ptr(), x.data_ptr(), out.data_ptr(), 0.0, 1, s) == 0      # warm call
torch.cuda.synchronize()
free0, count0 = torch.cuda.mem_get_info()[0], so.launch_count()
for n in (1 << 22, 12345, 1 << 20):
    assert L.stream_dot_noalloc_f64(x.data_ptr(), x.data_ptr(), out.data_ptr(), 0.0, n, s) == 0
    torch.cuda.synchronize()
    assert out.item() == float(n)
assert torch.cuda.mem_get_info()[0] == free0, "free device memory changed across no-allocation calls"
assert so.launch_count() == count0 + 3
so.dot(x, x, out)                                  # the regular Dot creates its workspace now
torch.cuda.synchronize()
assert torch.cuda.mem_get_info()[0] < free0, "the regular Dot's workspace existed already"
print("ok")
"""
    import os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", code], cwd=root, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "ok" in r.stdout, r.stdout + r.stderr
