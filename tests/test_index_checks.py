"""The index-checking build (libstreamops_checked.so, -DSTREAMOPS_CHECK_INDICES): a debugging aid that
stands in for an external memory checker. On a GPU the register-vector kernels run through it over
sizes with ragged ends and shifted pointers and must produce the oracle's results with no access
refused; the checker itself is exercised by a kernel that only ASKS about an access that does not
fit (no memory is touched), after which the record must name that access. Runs in a child process,
because the library to load is chosen by an environment variable at import time."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import numpy as np, torch, oracle
from paper_2510_00932_b200 import streamops as so
assert so.LIB_PATH.endswith("libstreamops_checked.so")
so.lib()
assert so.index_violation() is None
rng = np.random.Generator(np.random.PCG64(7))
for t, npdt in (("f64", np.float64), ("f32", np.float32)):
    for n in (1, 5, 1023, 4096, 70001, (1 << 20) + 7, 3 * 148 * 512 * 8 + 4099):
        for off in (0, 1, 3):
            x = rng.standard_normal(n + off).astype(npdt); y = rng.standard_normal(n + off).astype(npdt)
            dx, dy = torch.from_numpy(x).cuda()[off:], torch.from_numpy(y).cuda()[off:]
            out = torch.empty(n + off, dtype=dx.dtype, device="cuda")[off:]
            d = torch.zeros(1, dtype=dx.dtype, device="cuda")
            hx, hy = x[off:], y[off:]
            so.copy(dx, out); assert (out.cpu().numpy().view(np.uint8) == hx.view(np.uint8)).all()
            so.scale(dx, out, 0.4); assert (out.cpu().numpy() == oracle.scale(hx, 0.4)).all()
            so.add(dx, dy, out); assert (out.cpu().numpy() == oracle.add(hx, hy)).all()
            so.triad(dx, dy, out, 0.4); assert (out.cpu().numpy() == oracle.triad(hx, hy, 0.4)).all()
            for tun in (dict(pipeline=1, unroll=2), dict(pipeline=0, unroll=4), dict(pipeline=0, unroll=2, vec_bytes=16)):
                so.reset_tuning(); so.set_tuning("dot", t, **tun)
                so.dot(dx, dy, d)
                w = oracle.dot(hx, hy); s = oracle.dot_abs(hx, hy)
                assert abs(d.item() - w) <= (1e-12 if t == "f64" else 1e-5) * max(abs(w), 1e-3 * s), (t, n, off, tun)
            so.reset_tuning()
    assert so.index_violation() is None, "an access was refused on a correct run"
# the checker itself: an access of 32 bytes that ends 7 bytes past an array of 4096 bytes is refused and
# recorded; the last access that fits is accepted
assert so.index_selftest(4096 - 25, 32, 4096) == 2
v = so.index_violation()
assert v == {"where": 99, "offset": 4096 - 25, "limit": 4096}, v
assert so.index_violation() is None                      # reading the record clears it
assert so.index_selftest(4096 - 32, 32, 4096) == 3 and so.index_violation() is None
print("checked build ok")
"""


def _checked_library():
    from paper_2510_00932_b200 import build
    return build.build(checked=True)


def test_both_builds_export_the_index_check_entry_points_and_the_ordinary_one_declines():
    import ctypes
    from paper_2510_00932_b200 import build, streamops as so
    for path in (build.build(), _checked_library()):
        L = ctypes.CDLL(path)
        assert hasattr(L, "streamops_index_violation") and hasattr(L, "streamops_index_selftest")
    L = ctypes.CDLL(build.build())
    assert L.streamops_index_violation(None, None, None) == -7       # not a checking build
    assert L.streamops_index_selftest(0, 8, 64) == -7


@pytest.mark.gpu
def test_checked_build_runs_the_kernels_clean_and_its_checker_reports_a_planted_question():
    env = dict(os.environ, STREAMOPS_LIBRARY=_checked_library(), PYTHONPATH=ROOT)
    r = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "checked build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
