import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def bits(arr):
    """Raw bit patterns of a float array, for bit-exact comparison."""
    import numpy as np
    return arr.view(np.uint64 if arr.dtype.itemsize == 8 else np.uint32)


def assert_bits_equal(got, want, what=""):
    """Bit-exact equality, except that any NaN matches any NaN (payload propagation differs
    between processors); use a raw comparison where payloads must survive."""
    import numpy as np
    assert got.dtype == want.dtype and got.shape == want.shape, what
    both_nan = np.isnan(got) & np.isnan(want)
    same = (bits(got) == bits(want)) | both_nan
    if not same.all():
        i = int(np.flatnonzero(~same)[0])
        raise AssertionError(
            f"{what}: {int((~same).sum())} of {got.size} elements differ; first at {i}: "
            f"got {got[i]!r} ({int(bits(got)[i]):#x}) want {want[i]!r} ({int(bits(want)[i]):#x})")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle
