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

// Fixed-order sum of partials[0..count-1] by one block; thread 0 writes (T)total to out. The caller
// makes sure (with a barrier) that nobody is still reading warp_part from an earlier block_sum.
template <typename T>
__device__ __forceinline__ void finish(const double *partials, unsigned count, T *out, double *warp_part) {
    double acc = 0.0;
    for (unsigned b = threadIdx.x; b < count; b += blockDim.x) acc += __ldcg(partials + b);
    const double total = block_sum(acc, warp_part);
    if (threadIdx.x == 0) out[0] = (T)total;
}

// Arrival at a slot's ticket: one atomic add with release and acquire semantics. The release half
// publishes the partial sum this thread stored just before; the acquire half of the LAST arrival
// makes every earlier block's partial sum visible to it (the adds form one release sequence), so no
// separate fences are needed.
__device__ __forceinline__ unsigned arrive(unsigned long long *ticket_word) {
    unsigned t;
    asm volatile("atom.add.acq_rel.gpu.u32 %0, [%1], 1;" : "=r"(t) : "l"(ticket_word) : "memory");
    return t;
}
// Last act of the block that finishes a Dot: ticket back to zero and the call's sequence number in the
// word's high half, in one store (see DotScratch).
__device__ __forceinline__ void rearm(unsigned long long *ticket_word, unsigned seq) {
    *ticket_word = (unsigned long long)seq << 32;
}

// Publishes this block's partial sum; in the single-launch form the block that arrives last at
// the ticket then folds all partials (in block-index order) and re-arms the ticket.
template <typename T, bool SINGLE_LAUNCH>
__device__ __forceinline__ void publish_partial(double bsum, double *partials, unsigned long long *ticket, T *out,
                                                double *warp_part, bool *is_last, unsigned seq) {
    if (threadIdx.x == 0) partials[blockIdx.x] = bsum;
    if constexpr (SINGLE_LAUNCH) {
        if (threadIdx.x == 0) *is_last = (arrive(ticket) == gridDim.x - 1);
        __syncthreads();
        if (*is_last) {
            finish<T>(partials, gridDim.x, out, warp_part);
            if (threadIdx.x == 0) rearm(ticket, seq);
        }
    }
}

}  // namespace streamops
