"""Helpers for the GPU parity tests: guarded device buffers and tuning sets."""
import numpy as np

GUARD = 64          # guard elements either side of every device buffer
SENTINEL = {np.dtype(np.float64): 0x7FF8DEADBEEF0001, np.dtype(np.float32): 0x7FC0BEEF}


def _uint(dtype):
    return np.uint64 if np.dtype(dtype).itemsize == 8 else np.uint32


class Guarded:
    """A device tensor of n elements starting `offset` elements past an aligned base, with
    sentinel-filled guard regions either side that must survive every kernel."""

    def __init__(self, torch, host=None, n=None, dtype=None, offset=0):
        dtype = np.dtype(host.dtype if host is not None else dtype)
        n = host.size if host is not None else n
        self.n, self.offset, self.dtype = n, offset, dtype
        total = GUARD + offset + n + GUARD
        raw = np.full(total, SENTINEL[dtype], dtype=_uint(dtype)).view(dtype)
        if host is not None:
            raw[GUARD + offset:GUARD + offset + n] = host
        self.full = torch.from_numpy(raw).cuda()
        self.t = self.full[GUARD + offset:GUARD + offset + n]

    def host(self):
        return self.t.cpu().numpy()

    def guards_intact(self):
        full = self.full.cpu().numpy().view(_uint(self.dtype))
        lo = full[:GUARD + self.offset]
        hi = full[GUARD + self.offset + self.n:]
        s = SENTINEL[self.dtype]
        return bool((lo == s).all() and (hi == s).all())


# launch shapes that every parity case is repeated under (beside the defaults)
VEC_TUNINGS = [
    dict(kind=0, vec_bytes=16, unroll=1, threads=128, blocks_per_sm=1, policy=0, contiguous=0),
    dict(kind=0, vec_bytes=16, unroll=4, threads=256, blocks_per_sm=0, policy=1, contiguous=0),
    dict(kind=0, vec_bytes=32, unroll=1, threads=256, blocks_per_sm=2, policy=2, contiguous=1),
    dict(kind=0, vec_bytes=32, unroll=2, threads=512, blocks_per_sm=4, policy=3, contiguous=0),
    dict(kind=0, vec_bytes=32, unroll=4, threads=512, blocks_per_sm=1, policy=4, contiguous=1),
    dict(kind=0, vec_bytes=16, unroll=2, threads=512, blocks_per_sm=8, policy=4, contiguous=0),
    dict(kind=0, vec_bytes=32, unroll=2, threads=128, blocks_per_sm=0, policy=5, contiguous=0, reverse=1, pdl=1),
    dict(kind=0, vec_bytes=16, unroll=4, threads=256, blocks_per_sm=3, policy=6, contiguous=1, reverse=1),
    dict(kind=0, vec_bytes=32, unroll=4, threads=256, blocks_per_sm=0, policy=7, contiguous=0, reverse=0, keep_mib=1),
    dict(kind=0, vec_bytes=16, unroll=2, threads=128, blocks_per_sm=2, policy=8, contiguous=0, reverse=1, keep_mib=0),
    # the rolling-slot Dot kernel (the elementwise kernels ignore `pipeline`)
    dict(kind=0, vec_bytes=32, unroll=2, threads=512, blocks_per_sm=0, policy=4, contiguous=0, pipeline=1),
    dict(kind=0, vec_bytes=32, unroll=4, threads=256, blocks_per_sm=1, policy=0, contiguous=0, pipeline=1),
    dict(kind=0, vec_bytes=32, unroll=2, threads=128, blocks_per_sm=3, policy=4, contiguous=0, pipeline=1, two_pass=1),
]
BULK_TUNINGS = [
    dict(kind=1, threads=128, blocks_per_sm=1, chunk_bytes=1024, stages=2),
    dict(kind=1, threads=256, blocks_per_sm=1, chunk_bytes=16384, stages=6),
    dict(kind=1, threads=512, blocks_per_sm=2, chunk_bytes=8192, stages=4),
    dict(kind=1, threads=256, blocks_per_sm=1, chunk_bytes=4112, stages=3),
]
