// Fixed-order reductions shared by the Dot kernels: every fold below has an order that depends
// only on thread and block indices, so results are bitwise repeatable.
#pragma once
#include <cuda_runtime.h>

namespace streamops {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// Sum over the block, returned to every thread of warp 0 (valid in thread 0).
__device__ __forceinline__ double block_sum(double v, double *warp_part) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nwarps = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    if (lane == 0) warp_part[warp] = v;
    __syncthreads();
    double r = 0.0;
    if (warp == 0) {
        r = lane < nwarps ? warp_part[lane] : 0.0;
        r = warp_sum(r);
    }
    return r;
}

template <typename T> __device__ __forceinline__ double widen(T v) { return (double)v; }

// Fixed-order sum of partials[0..count-1] by one block; thread 0 writes (T)total to out.
template <typename T>
__device__ __forceinline__ void finish(const double *partials, unsigned count, T *out, double *warp_part) {
    double acc = 0.0;
    for (unsigned b = threadIdx.x; b < count; b += blockDim.x) acc += __ldcg(partials + b);
    __syncthreads();                      // warp_part is reused
    const double total = block_sum(acc, warp_part);
    if (threadIdx.x == 0) out[0] = (T)total;
}

// Last act of the thread that finishes a Dot: after everything it read or wrote in the slot's
// scratch, it publishes the call's sequence number, which tells the host (when it needs to know)
// that the slot is free for another stream.
__device__ __forceinline__ void mark_done(unsigned *done, unsigned seq) {
    if (done) {
        __threadfence();
        *done = seq;
    }
}

// Publishes this block's partial sum; in the single-launch form the block that arrives last at
// the ticket then folds all partials (in block-index order) and re-arms the ticket.
template <typename T, bool SINGLE_LAUNCH>
__device__ __forceinline__ void publish_partial(double bsum, double *partials, unsigned *ticket, T *out,
                                                double *warp_part, bool *is_last, unsigned *done, unsigned seq) {
    if (threadIdx.x == 0) partials[blockIdx.x] = bsum;
    if constexpr (SINGLE_LAUNCH) {
        if (threadIdx.x == 0) {
            __threadfence();                                  // partial visible before the ticket
            const unsigned t = atomicAdd(ticket, 1u);
            *is_last = (t == gridDim.x - 1);
        }
        __syncthreads();
        if (*is_last) {
            __threadfence();
            finish<T>(partials, gridDim.x, out, warp_part);
            if (threadIdx.x == 0) {
                *ticket = 0u;                                 // ready for the next call
                mark_done(done, seq);
            }
        }
    }
}

}  // namespace streamops
