"""ctypes binding of libstreamops: argument marshalling only.

Each function below forwards to the C entry point of the same name (see include/streamops.h).
Tensors supply device pointers, ``torch.cuda.current_stream()`` supplies the stream; every step
of the computation runs inside the library's CUDA kernels. There is no fallback: if the shared
library is missing or a call returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
# STREAMOPS_LIBRARY selects another build of the same library, e.g. the index-checking one
# (libstreamops_checked.so, written by `python -m paper_2510_00932_b200.build --checked`)
LIB_PATH = os.environ.get("STREAMOPS_LIBRARY") or os.path.join(_HERE, "libstreamops.so")

OPS = ("copy", "scale", "add", "triad", "dot")
OP_CODE = {name: i for i, name in enumerate(OPS)}
DTYPE_CODE = {"f32": 0, "f64": 1}
# arrays moved per element, counted the standard STREAM way
ARRAYS_MOVED = {"copy": 2, "scale": 2, "add": 3, "triad": 3, "dot": 2}


class StreamopsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"libstreamops status {status}: {message}")
        self.status = status


class Tuning(ctypes.Structure):
    """Mirror of streamops_tuning_t."""
    _fields_ = [(n, ctypes.c_int) for n in (
        "kind", "vec_bytes", "unroll", "threads", "blocks_per_sm", "policy", "contiguous",
        "chunk_bytes", "stages", "two_pass", "reverse", "pdl", "keep_mib", "compensated", "pipeline")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libstreamops.so (built in-tree by ``build.py``); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with "
                              "`python -m paper_2510_00932_b200.build` (needs nvcc)")
        L = ctypes.CDLL(LIB_PATH)
        vp, dbl, sz, ci = ctypes.c_void_p, ctypes.c_double, ctypes.c_size_t, ctypes.c_int
        for t in ("f32", "f64"):
            for name in ("copy", "scale"):
                f = getattr(L, f"stream_{name}_{t}")
                f.argtypes, f.restype = [vp, vp, dbl, sz, vp], ci
            for name in ("add", "triad", "dot"):
                f = getattr(L, f"stream_{name}_{t}")
                f.argtypes, f.restype = [vp, vp, vp, dbl, sz, vp], ci
            f = getattr(L, f"streamops_chain_host_{t}")
            f.argtypes, f.restype = [vp, vp, vp, dbl, sz, vp], ci
            f = getattr(L, f"streamops_chain_{t}")
            f.argtypes, f.restype = [vp, vp, vp, vp, dbl, sz, vp], ci
        L.stream_dot_wide_f32.argtypes, L.stream_dot_wide_f32.restype = [vp, vp, vp, dbl, sz, vp], ci
        for t in ("f32", "f64"):
            f = getattr(L, f"stream_fold_{t}")
            f.argtypes, f.restype = [vp, vp, dbl, sz, vp], ci
        L.stream_dot_timeline_f64.argtypes = [vp, vp, vp, sz, vp, vp, ctypes.POINTER(ctypes.c_uint)]
        L.stream_dot_timeline_f64.restype = ci
        L.stream_dot_noalloc_f64.argtypes, L.stream_dot_noalloc_f64.restype = [vp, vp, vp, dbl, sz, vp], ci
        L.shmem_mix_u32.argtypes, L.shmem_mix_u32.restype = [vp, vp, ctypes.c_uint, sz, vp], ci
        L.streamops_set_shmem_width.argtypes, L.streamops_set_shmem_width.restype = [ci], ci
        L.streamops_get_shmem_width.argtypes, L.streamops_get_shmem_width.restype = [], ci
        L.streamops_init.argtypes, L.streamops_init.restype = [ci], ci
        L.streamops_set_host_piece_mib.argtypes, L.streamops_set_host_piece_mib.restype = [ci], ci
        L.streamops_shutdown.argtypes, L.streamops_shutdown.restype = [], ci
        L.streamops_set_tuning.argtypes, L.streamops_set_tuning.restype = [ci, ci, ctypes.POINTER(Tuning)], ci
        L.streamops_get_tuning.argtypes, L.streamops_get_tuning.restype = [ci, ci, ctypes.POINTER(Tuning)], ci
        L.streamops_reset_tuning.argtypes, L.streamops_reset_tuning.restype = [], ci
        L.streamops_policy_name.argtypes, L.streamops_policy_name.restype = [ci], ctypes.c_char_p
        L.streamops_check.argtypes, L.streamops_check.restype = [vp], ci
        L.streamops_set_wait_limit.argtypes, L.streamops_set_wait_limit.restype = [ctypes.c_uint], ci
        ullp = ctypes.POINTER(ctypes.c_ulonglong)
        L.streamops_index_violation.argtypes, L.streamops_index_violation.restype = [ctypes.POINTER(ci), ullp, ullp], ci
        L.streamops_index_selftest.argtypes, L.streamops_index_selftest.restype = [ctypes.c_ulonglong] * 3, ci
        L.streamops_status_string.argtypes, L.streamops_status_string.restype = [ci], ctypes.c_char_p
        L.streamops_last_cuda_error.argtypes, L.streamops_last_cuda_error.restype = [], ci
        L.streamops_launch_count.argtypes, L.streamops_launch_count.restype = [], ctypes.c_ulonglong
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().streamops_status_string(int(status)).decode()


def _raise(status: int):
    if status != 0:
        msg = status_string(status)
        if status == 4:
            msg += f" [cudaError {lib().streamops_last_cuda_error()}]"
        raise StreamopsError(status, msg)


_SUFFIX = None            # torch dtype -> "f32" / "f64", filled on first use
_raw_stream = None        # fast accessor of the current stream's handle
_current_device = None    # fast accessor of the current CUDA device index


def _suffix(t) -> str:
    global _SUFFIX
    if _SUFFIX is None:
        import torch
        _SUFFIX = {torch.float64: "f64", torch.float32: "f32"}
    try:
        return _SUFFIX[t.dtype]
    except KeyError:
        raise TypeError(f"libstreamops handles float32 and float64 tensors, got {t.dtype}") from None


def _marshal(*tensors):
    """Common dtype suffix and the current stream handle of the tensors' device. Kept lean: at
    L2-resident sizes a kernel lasts a few microseconds and this code is what the host spends."""
    global _raw_stream, _current_device
    first = tensors[0]
    suf = _suffix(first)
    dev = first.get_device()
    for t in tensors:
        if not t.is_cuda:
            raise ValueError("libstreamops operates on CUDA tensors")
        if t.dim() != 1 or not t.is_contiguous():
            raise ValueError("libstreamops operates on contiguous 1-D tensors")
        if t.dtype != first.dtype or t.get_device() != dev:
            raise ValueError("all tensors of one call share dtype and device")
    if _raw_stream is None:
        import torch
        _raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None) or (
            lambda d: torch.cuda.current_stream(d).cuda_stream)
        _current_device = getattr(torch._C, "_cuda_getDevice", None) or torch.cuda.current_device
    # the library takes its per-device state (Dot workspace, SM count) from the CURRENT device
    if dev != _current_device():
        raise ValueError(f"tensors live on cuda:{dev} but the current device is cuda:{_current_device()}; "
                         "make the tensors' device current (torch.cuda.device) around the call")
    return suf, _raw_stream(dev)


def copy(x, out, scalar: float = 0.0):
    """out[i] = x[i] (stream_copy_*)."""
    suf, stream = _marshal(x, out)
    if out.numel() != x.numel():
        raise ValueError("length mismatch")
    _raise(getattr(lib(), f"stream_copy_{suf}")(x.data_ptr(), out.data_ptr(), float(scalar), x.numel(), stream))
    return out


def scale(x, out, scalar: float):
    """out[i] = RN(s * x[i]) (stream_scale_*)."""
    suf, stream = _marshal(x, out)
    if out.numel() != x.numel():
        raise ValueError("length mismatch")
    _raise(getattr(lib(), f"stream_scale_{suf}")(x.data_ptr(), out.data_ptr(), float(scalar), x.numel(), stream))
    return out


def add(x, y, out, scalar: float = 0.0):
    """out[i] = RN(x[i] + y[i]) (stream_add_*)."""
    suf, stream = _marshal(x, y, out)
    if not (out.numel() == x.numel() == y.numel()):
        raise ValueError("length mismatch")
    _raise(getattr(lib(), f"stream_add_{suf}")(x.data_ptr(), y.data_ptr(), out.data_ptr(), float(scalar), x.numel(), stream))
    return out


def triad(x, y, out, scalar: float):
    """out[i] = RN(x[i] + RN(s * y[i])) (stream_triad_*)."""
    suf, stream = _marshal(x, y, out)
    if not (out.numel() == x.numel() == y.numel()):
        raise ValueError("length mismatch")
    _raise(getattr(lib(), f"stream_triad_{suf}")(x.data_ptr(), y.data_ptr(), out.data_ptr(), float(scalar), x.numel(), stream))
    return out


def dot(x, y, out, scalar: float = 0.0):
    """out[0] = (T) sum x[i]*y[i]; out is a one-element device tensor (stream_dot_*)."""
    suf, stream = _marshal(x, y, out)
    if x.numel() != y.numel() or out.numel() != 1:
        raise ValueError("dot takes two equal-length inputs and a one-element output")
    _raise(getattr(lib(), f"stream_dot_{suf}")(x.data_ptr(), y.data_ptr(), out.data_ptr(), float(scalar), x.numel(), stream))
    return out


def dot_wide(x, y, out64):
    """out64[0] = the double-precision sum of x[i]*y[i] before any rounding to the element type;
    out64 is a one-element float64 device tensor (stream_dot_wide_f32 / stream_dot_f64)."""
    import torch
    suf, stream = _marshal(x, y)
    if out64.is_cuda and out64.get_device() != x.get_device():
        raise ValueError("all tensors of one call share a device")
    if x.numel() != y.numel() or out64.numel() != 1 or out64.dtype != torch.float64 or not out64.is_cuda:
        raise ValueError("dot_wide takes two equal-length inputs and a one-element float64 device output")
    f = lib().stream_dot_f64 if suf == "f64" else lib().stream_dot_wide_f32
    _raise(f(x.data_ptr(), y.data_ptr(), out64.data_ptr(), 0.0, x.numel(), stream))
    return out64


def fold(partials, out):
    """out[0] = the float64 partials added left to right, rounded once to out's type (stream_fold_*)."""
    import torch
    if partials.dtype != torch.float64 or not partials.is_cuda or not partials.is_contiguous() or partials.dim() != 1:
        raise ValueError("fold takes a contiguous 1-D float64 device tensor of partial sums")
    suf, stream = _marshal(out)
    if out.numel() != 1 or partials.get_device() != out.get_device():
        raise ValueError("fold writes one element on the device that holds the partial sums")
    _raise(getattr(lib(), f"stream_fold_{suf}")(partials.data_ptr(), out.data_ptr(), 0.0, partials.numel(), stream))
    return out


TIMELINE_MAX_BLOCKS = 1024


def dot_timeline(x, y, out, stamps) -> int:
    """The default fp64 Dot with three global-timer stamps per block written to the int64 device tensor
    `stamps` (at least 3 * TIMELINE_MAX_BLOCKS entries); returns the number of blocks launched."""
    import torch
    suf, stream = _marshal(x, y, out)
    if suf != "f64" or x.numel() != y.numel() or out.numel() != 1:
        raise ValueError("dot_timeline takes two equal-length float64 inputs and a one-element output")
    if stamps.dtype != torch.int64 or not stamps.is_cuda or stamps.numel() < 3 * TIMELINE_MAX_BLOCKS or not stamps.is_contiguous():
        raise ValueError("stamps is a contiguous int64 CUDA tensor of at least 3 * TIMELINE_MAX_BLOCKS entries")
    blocks = ctypes.c_uint(0)
    _raise(lib().stream_dot_timeline_f64(x.data_ptr(), y.data_ptr(), out.data_ptr(), x.numel(), stream, stamps.data_ptr(),
                                         ctypes.byref(blocks)))
    return int(blocks.value)


DOT_NOALLOC_MAX_N = 1 << 28


def dot_noalloc(x, y, out, scalar: float = 0.0):
    """fp64 Dot through stream_dot_noalloc_f64: for callers that cannot allocate device memory
    (the whole device already belongs to a pool, or the allocator's lock and implicit
    synchronisation are off limits where the result is needed). The partial sums sit in a fixed
    array inside the library, so n is limited to DOT_NOALLOC_MAX_N and calls that overlap in time
    on one GPU race; make the first call on a device outside stream capture."""
    suf, stream = _marshal(x, y, out)
    if suf != "f64":
        raise TypeError("the no-allocation Dot is fp64 only")
    if x.numel() != y.numel() or out.numel() != 1:
        raise ValueError("dot takes two equal-length inputs and a one-element output")
    _raise(lib().stream_dot_noalloc_f64(x.data_ptr(), y.data_ptr(), out.data_ptr(), float(scalar), x.numel(), stream))
    return out


def shmem_mix(x, out, rounds: int):
    """out = x after `rounds` rounds of the shared-memory exchange (shmem_mix_u32): int32/uint32
    CUDA tensors of equal length, treated as raw 32-bit words."""
    import torch
    for t in (x, out):
        if not t.is_cuda or t.dim() != 1 or not t.is_contiguous() or t.element_size() != 4 or t.is_floating_point():
            raise ValueError("shmem_mix operates on contiguous 1-D CUDA tensors of 32-bit integers")
    if x.numel() != out.numel() or x.get_device() != out.get_device():
        raise ValueError("length or device mismatch")
    if not 0 <= int(rounds) < 2 ** 32:
        raise ValueError("rounds out of range")
    if x.get_device() != torch.cuda.current_device():
        raise ValueError("make the tensors' device current around the call")
    stream = torch.cuda.current_stream(x.get_device()).cuda_stream
    _raise(lib().shmem_mix_u32(x.data_ptr(), out.data_ptr(), int(rounds), x.numel(), stream))
    return out


def set_shmem_width(width_bytes: int):
    _raise(lib().streamops_set_shmem_width(int(width_bytes)))


def chain(a, b, c, dot_out, scalar: float):
    """One pass of the five kernels over device tensors a, b, c in the STREAM dataflow:
    c <- a; b <- s*c; c <- a+b; a <- b+s*c; dot_out <- dot(a, b) (streamops_chain_*: one library
    call, five asynchronous launches)."""
    suf, stream = _marshal(a, b, c, dot_out)
    if not (a.numel() == b.numel() == c.numel()) or dot_out.numel() != 1:
        raise ValueError("chain takes three equal-length arrays and a one-element output")
    _raise(getattr(lib(), f"streamops_chain_{suf}")(a.data_ptr(), b.data_ptr(), c.data_ptr(), dot_out.data_ptr(),
                                                   float(scalar), a.numel(), stream))


def chain_host(a, b, c, scalar: float):
    """The same pass over three HOST numpy arrays, updated in place through
    streamops_chain_host_*; returns the dot product. Copies in both directions happen inside
    the library call."""
    import numpy as np
    suf = {np.dtype(np.float64): "f64", np.dtype(np.float32): "f32"}[a.dtype]
    for arr in (a, b, c):
        if arr.dtype != a.dtype or arr.shape != a.shape or arr.ndim != 1 or not arr.flags.c_contiguous:
            raise ValueError("chain_host takes three contiguous 1-D arrays of one dtype and length")
    res = np.zeros(1, dtype=a.dtype)
    _raise(getattr(lib(), f"streamops_chain_host_{suf}")(a.ctypes.data, b.ctypes.data, c.ctypes.data,
                                                        float(scalar), a.size, res.ctypes.data))
    return res[0]


def set_host_piece_mib(mib: int):
    _raise(lib().streamops_set_host_piece_mib(int(mib)))


def init(device: int = 0):
    _raise(lib().streamops_init(int(device)))


def shutdown():
    _raise(lib().streamops_shutdown())


def get_tuning(op: str, dtype: str) -> Tuning:
    t = Tuning()
    _raise(lib().streamops_get_tuning(OP_CODE[op], DTYPE_CODE[dtype], ctypes.byref(t)))
    return t


def set_tuning(op: str, dtype: str, **fields) -> Tuning:
    """Overrides fields of the (op, dtype) tuning; returns the tuning now in force."""
    t = get_tuning(op, dtype)
    for k, v in fields.items():
        if not hasattr(t, k):
            raise KeyError(k)
        setattr(t, k, int(v))
    _raise(lib().streamops_set_tuning(OP_CODE[op], DTYPE_CODE[dtype], ctypes.byref(t)))
    return t


def reset_tuning():
    _raise(lib().streamops_reset_tuning())


def policy_name(policy: int) -> str:
    return lib().streamops_policy_name(int(policy)).decode()


def check(stream=None):
    """Synchronises the stream and raises if a bounded wait inside a kernel gave up."""
    import torch
    s = (stream or torch.cuda.current_stream()).cuda_stream
    _raise(lib().streamops_check(s))


def set_wait_limit(tries: int):
    """Attempts a wait inside the bulk-copy pipelines makes before giving up (0 = default)."""
    _raise(lib().streamops_set_wait_limit(int(tries)))


def index_violation():
    """Index-checking builds: None if no access was refused since the last call, else a dict with the
    kind of access, its byte offset and the array's byte length. Raises in an ordinary build."""
    where, off, lim = ctypes.c_int(0), ctypes.c_ulonglong(0), ctypes.c_ulonglong(0)
    rc = lib().streamops_index_violation(ctypes.byref(where), ctypes.byref(off), ctypes.byref(lim))
    if rc < 0:
        _raise(-rc)
    return None if rc == 0 else {"where": where.value, "offset": off.value, "limit": lim.value}


def index_selftest(offset: int, width: int, limit: int) -> int:
    rc = lib().streamops_index_selftest(int(offset), int(width), int(limit))
    if rc < 0:
        _raise(-rc)
    return rc


def launch_count() -> int:
    return int(lib().streamops_launch_count())
