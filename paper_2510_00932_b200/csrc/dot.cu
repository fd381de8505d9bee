// Dot kernels (Table 1 of the paper, "Dot"): out[0] = (T) sum_i x[i] * y[i].
//
// Pass 1 streams x and y exactly like the elementwise kernels (tiles of blockDim.x * U vectors,
// tiles interleaved across a persistent grid) and keeps U double-precision accumulators per
// thread; float inputs are widened first, so every product is exact. The accumulators are
// folded in a fixed order: per thread (u = 0..U-1), per warp (xor-shuffle tree), per block
// (shared memory, warp 0 folds the warp sums), giving partials[blockIdx.x].
//
// A second pass-1 form, the rolling-slot kernel, gives each thread S slots of one vector of x and one
// of y: the oldest slot is folded into its accumulator and reloaded at once, so S - 1 loads per array
// stay in flight per thread all the time instead of all of them draining before the next tile is
// requested. Slot s of thread t owns tiles b + (s + k S) G (k = 0, 1, ...) of block b: still a fixed
// function of n and the launch shape.
//
// Pass 2 sums partials[0..G-1] with one block in a fixed order (thread t takes t, t + B, ... in
// sequence, then the same warp/block tree). It runs either as its own launch or inside pass 1
// by whichever block arrives last at an atomic ticket: the ticket only elects WHO does pass 2,
// the order of the additions is by block index, so the bits of the result never depend on
// block scheduling, on the stream, or on what else the GPU is running.
#include "indexcheck.cuh"
#include "internal.cuh"
#include "memops.cuh"
#include "reduce.cuh"

namespace streamops {

namespace {

template <typename T, int VB>
__device__ __forceinline__ double fold_vec(double acc, const Vec<VB> &xv, const Vec<VB> &yv) {
    constexpr int EPV = VB / (int)sizeof(T);
#pragma unroll
    for (int e = 0; e < EPV; ++e)
        acc = fma(widen<T>(Lanes<T>::get(xv.w, e)), widen<T>(Lanes<T>::get(yv.w, e)), acc);
    return acc;
}

template <typename T, int VB, int U, int POL, bool SINGLE_LAUNCH>
__global__ void __launch_bounds__(kMaxThreads)
dot_pass1_kernel(const T *x, const T *y, size_t n, double *partials, unsigned long long *ticket, T *out, int reverse,
                 unsigned seq) {
    constexpr int EPV = VB / (int)sizeof(T);
    __shared__ double warp_part[32];
    __shared__ bool is_last;
    grid_dependency_sync();
    const char *xb = reinterpret_cast<const char *>(x);
    const char *yb = reinterpret_cast<const char *>(y);
    const uint64_t l2pol = make_l2_policies<POL>().ld;

    const size_t nvec = n / EPV;
    const size_t tile_vecs = (size_t)blockDim.x * U;
    const size_t ntiles = nvec / tile_vecs;
    double acc[U];
#pragma unroll
    for (int u = 0; u < U; ++u) acc[u] = 0.0;

    for (size_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const size_t v0 = (reverse ? ntiles - 1 - tile : tile) * tile_vecs + threadIdx.x;
        Vec<VB> xv[U], yv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
#ifdef STREAMOPS_CHECK_INDICES
            xv[u] = Vec<VB>{};                         // an access a checking build refuses contributes zero
#endif
            if (index_ok((v0 + (size_t)u * blockDim.x) * VB, VB, n * sizeof(T), W_DOT_LOAD_X))
                ldg<POL>(xv[u], xb + (v0 + (size_t)u * blockDim.x) * VB, l2pol);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
#ifdef STREAMOPS_CHECK_INDICES
            yv[u] = Vec<VB>{};
#endif
            if (index_ok((v0 + (size_t)u * blockDim.x) * VB, VB, n * sizeof(T), W_DOT_LOAD_Y))
                ldg<POL>(yv[u], yb + (v0 + (size_t)u * blockDim.x) * VB, l2pol);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) acc[u] = fold_vec<T, VB>(acc[u], xv[u], yv[u]);
    }
    if (blockIdx.x == (unsigned)(ntiles % gridDim.x)) {      // ragged end, one block
        for (size_t v = ntiles * tile_vecs + threadIdx.x; v < nvec; v += blockDim.x) {
            Vec<VB> xv, yv;
            ldg<0>(xv, xb + v * VB, 0);
            ldg<0>(yv, yb + v * VB, 0);
            acc[0] = fold_vec<T, VB>(acc[0], xv, yv);
        }
        const size_t i = nvec * EPV + threadIdx.x;
        if (i < n) acc[0] = fma(widen<T>(x[i]), widen<T>(y[i]), acc[0]);
    }
    double tsum = acc[0];
#pragma unroll
    for (int u = 1; u < U; ++u) tsum += acc[u];
    const double bsum = block_sum(tsum, warp_part);

    publish_partial<T, SINGLE_LAUNCH>(bsum, partials, ticket, out, warp_part, &is_last, seq);
}

__device__ __forceinline__ unsigned long long global_nanoseconds() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Rolling-slot pass 1 (see the file comment). A tile is blockDim.x vectors: one vector per thread.
// With TRACE (the timeline entry point only) thread 0 of every block stores three global-timer readings
// into stamps[3 * blockIdx.x ..]: after the wait for the previous kernel, after its last fold, and at the
// block's end (for the finishing block: after the final fold and the write of the result).
template <typename T, int VB, int S, int POL, bool SINGLE_LAUNCH, bool TRACE = false>
__global__ void __launch_bounds__(kMaxThreads, S <= 2 ? 2 : 1)
dot_roll_kernel(const T *x, const T *y, size_t n, double *partials, unsigned long long *ticket, T *out, unsigned seq,
                unsigned long long *stamps) {
    constexpr int EPV = VB / (int)sizeof(T);
    __shared__ double warp_part[32];
    __shared__ bool is_last;
    grid_dependency_sync();
    if constexpr (TRACE) {
        if (threadIdx.x == 0) stamps[3 * blockIdx.x] = global_nanoseconds();
    }
    const char *xb = reinterpret_cast<const char *>(x);
    const char *yb = reinterpret_cast<const char *>(y);
    const uint64_t l2pol = make_l2_policies<POL>().ld;

    const size_t nvec = n / EPV;
    const size_t ntiles = nvec / blockDim.x;
    const size_t G = gridDim.x;
    // byte offsets: a slot's vector of tile k sits at k * tile_bytes + threadIdx.x * VB, so "tile k exists"
    // is "offset < end"; slots of one round are slot_stride apart, rounds are round_stride apart
    const size_t tile_bytes = (size_t)blockDim.x * VB;
    const size_t end = ntiles * tile_bytes;
    const size_t slot_stride = G * tile_bytes;
    const size_t round_stride = (size_t)S * slot_stride;
    size_t off = (size_t)blockIdx.x * tile_bytes + (size_t)threadIdx.x * VB;
    double acc[S];
    Vec<VB> xv[S], yv[S];
#pragma unroll
    for (int s = 0; s < S; ++s) acc[s] = 0.0;
#pragma unroll
    for (int s = 0; s < S; ++s) {
        const size_t o = off + (size_t)s * slot_stride;
        if (o < end && index_ok(o, VB, n * sizeof(T), W_DOT_LOAD_X)) {
            ldg<POL>(xv[s], xb + o, l2pol);
            ldg<POL>(yv[s], yb + o, l2pol);
        }
    }
    for (; off < end; off += round_stride) {
#pragma unroll
        for (int s = 0; s < S; ++s) {
            const size_t o = off + (size_t)s * slot_stride;
            if (o < end) {
                acc[s] = fold_vec<T, VB>(acc[s], xv[s], yv[s]);
                const size_t next = o + round_stride;
                if (next < end && index_ok(next, VB, n * sizeof(T), W_DOT_LOAD_X)) {
                    ldg<POL>(xv[s], xb + next, l2pol);
                    ldg<POL>(yv[s], yb + next, l2pol);
                }
            }
        }
    }
    if (blockIdx.x == (unsigned)(ntiles % G)) {              // ragged end, one block
        for (size_t v = ntiles * blockDim.x + threadIdx.x; v < nvec; v += blockDim.x) {
            Vec<VB> xr, yr;
            ldg<0>(xr, xb + v * VB, 0);
            ldg<0>(yr, yb + v * VB, 0);
            acc[0] = fold_vec<T, VB>(acc[0], xr, yr);
        }
        const size_t i = nvec * EPV + threadIdx.x;
        if (i < n) acc[0] = fma(widen<T>(x[i]), widen<T>(y[i]), acc[0]);
    }
    double tsum = acc[0];
#pragma unroll
    for (int s = 1; s < S; ++s) tsum += acc[s];
    if constexpr (TRACE) {
        if (threadIdx.x == 0) stamps[3 * blockIdx.x + 1] = global_nanoseconds();
    }
    const double bsum = block_sum(tsum, warp_part);
    publish_partial<T, SINGLE_LAUNCH>(bsum, partials, ticket, out, warp_part, &is_last, seq);
    if constexpr (TRACE) {
        if (threadIdx.x == 0) stamps[3 * blockIdx.x + 2] = global_nanoseconds();
    }
}

template <typename T>
__global__ void __launch_bounds__(1024)
dot_pass2_kernel(const double *partials, unsigned count, T *out, unsigned long long *ticket, unsigned seq) {
    __shared__ double warp_part[32];
    finish<T>(partials, count, out, warp_part);
    if (threadIdx.x == 0) rearm(ticket, seq);
}

// Scalar pass 1 for pointers that are not 16-byte aligned: same structure, one element per load.
template <typename T, bool SINGLE_LAUNCH>
__global__ void __launch_bounds__(kMaxThreads)
dot_scalar_kernel(const T *x, const T *y, size_t n, double *partials, unsigned long long *ticket, T *out,
                  unsigned seq) {
    __shared__ double warp_part[32];
    __shared__ bool is_last;
    double acc = 0.0;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        acc = fma(widen<T>(x[i]), widen<T>(y[i]), acc);
    const double bsum = block_sum(acc, warp_part);
    publish_partial<T, SINGLE_LAUNCH>(bsum, partials, ticket, out, warp_part, &is_last, seq);
}

template <typename T, int VB, int U, bool SL>
cudaError_t launch_pol(const VecLaunch &c, const T *x, const T *y, size_t n, const DotScratch &s, T *out, cudaStream_t st) {
    switch (c.policy) {
#define STREAMOPS_CASE(P) case P: return launch_kernel(dot_pass1_kernel<T, VB, U, P, SL>, c.grid, c.threads, 0, st, c.pdl != 0, x, y, n, s.partials, s.ticket, out, c.reverse, s.seq);
        STREAMOPS_CASE(0) STREAMOPS_CASE(1) STREAMOPS_CASE(2) STREAMOPS_CASE(3) STREAMOPS_CASE(4) STREAMOPS_CASE(5) STREAMOPS_CASE(6)
#undef STREAMOPS_CASE
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

// The rolling-slot kernel loads with the evict-first set (4) or with plain loads (0).
template <typename T, int VB, bool SL>
cudaError_t launch_roll(const VecLaunch &c, const T *x, const T *y, size_t n, const DotScratch &s, T *out, cudaStream_t st) {
    const bool plain = c.policy == 0;
#define STREAMOPS_ROLL(S, P) launch_kernel(dot_roll_kernel<T, VB, S, P, SL>, c.grid, c.threads, 0, st, c.pdl != 0, x, y, n, s.partials, s.ticket, out, s.seq, (unsigned long long *)nullptr)
    if (c.unroll == 2) return plain ? STREAMOPS_ROLL(2, 0) : STREAMOPS_ROLL(2, 4);
    if (c.unroll == 4) return plain ? STREAMOPS_ROLL(4, 0) : STREAMOPS_ROLL(4, 4);
#undef STREAMOPS_ROLL
    return cudaErrorInvalidValue;
}

template <typename T, int VB, bool SL>
cudaError_t launch_unroll(const VecLaunch &c, const T *x, const T *y, size_t n, const DotScratch &s, T *out, cudaStream_t st) {
    switch (c.unroll) {
        case 1: return launch_pol<T, VB, 1, SL>(c, x, y, n, s, out, st);
        case 2: return launch_pol<T, VB, 2, SL>(c, x, y, n, s, out, st);
        case 4: return launch_pol<T, VB, 4, SL>(c, x, y, n, s, out, st);
        default: return cudaErrorInvalidValue;
    }
}

template <typename T, bool SL>
cudaError_t launch_pass1(const VecLaunch &c, const T *x, const T *y, size_t n, const DotScratch &s, T *out, cudaStream_t st) {
    if (c.vec_bytes == 32 && c.pipeline) return launch_roll<T, 32, SL>(c, x, y, n, s, out, st);
    if (c.vec_bytes == 32) return launch_unroll<T, 32, SL>(c, x, y, n, s, out, st);
    if (c.vec_bytes == 16) return launch_unroll<T, 16, SL>(c, x, y, n, s, out, st);
    dot_scalar_kernel<T, SL><<<c.grid, c.threads, 0, st>>>(x, y, n, s.partials, s.ticket, out, s.seq);
    return cudaGetLastError();
}

// Sequential left-to-right sum of count doubles by one thread: the order is the index order.
template <typename T>
__global__ void fold_kernel(const double *p, size_t count, T *out) {
    double acc = 0.0;
    for (size_t i = 0; i < count; ++i) acc += p[i];
    out[0] = (T)acc;
}

template <typename T>
cudaError_t launch_dot_t(const VecLaunch &c, bool two_pass, bool wide, const T *x, const T *y, void *out, size_t n,
                         const DotScratch &s, cudaStream_t st, int *launches) {
    if (c.grid > (unsigned)kMaxDotBlocks) return cudaErrorInvalidValue;
    if (wide) {                       // the unrounded double total: pass 1 as usual, pass 2 writes a double
        *launches = 2;
        cudaError_t e = launch_pass1<T, false>(c, x, y, n, s, (T *)nullptr, st);
        if (e != cudaSuccess) return e;
        dot_pass2_kernel<double><<<1, 1024, 0, st>>>(s.partials, c.grid, (double *)out, s.ticket, s.seq);
        return cudaGetLastError();
    }
    T *o = (T *)out;
    if (!two_pass) {
        *launches = 1;
        return launch_pass1<T, true>(c, x, y, n, s, o, st);
    }
    *launches = 2;
    cudaError_t e = launch_pass1<T, false>(c, x, y, n, s, o, st);
    if (e != cudaSuccess) return e;
    dot_pass2_kernel<T><<<1, 1024, 0, st>>>(s.partials, c.grid, o, s.ticket, s.seq);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_dot(int dtype, const VecLaunch &cfg, bool two_pass, bool wide, const void *x, const void *y,
                       void *out, size_t n, const DotScratch &scratch, cudaStream_t stream, int *launches) {
    if (dtype == DT_F64)
        return launch_dot_t<double>(cfg, two_pass, wide, (const double *)x, (const double *)y, out, n,
                                    scratch, stream, launches);
    return launch_dot_t<float>(cfg, two_pass, wide, (const float *)x, (const float *)y, out, n,
                               scratch, stream, launches);
}

// The default double-precision Dot (two rolling slots, evict-first loads, single launch) with time stamps.
cudaError_t launch_dot_timeline(const VecLaunch &c, const double *x, const double *y, double *out, size_t n,
                                const DotScratch &s, unsigned long long *stamps, cudaStream_t st) {
    return launch_kernel(dot_roll_kernel<double, 32, 2, 4, true, true>, c.grid, c.threads, 0, st, c.pdl != 0, x, y, n,
                         s.partials, s.ticket, out, s.seq, stamps);
}

cudaError_t launch_fold(int dtype, const double *partials, size_t count, void *out, cudaStream_t stream) {
    if (dtype == DT_F64) fold_kernel<double><<<1, 1, 0, stream>>>(partials, count, (double *)out);
    else fold_kernel<float><<<1, 1, 0, stream>>>(partials, count, (float *)out);
    return cudaGetLastError();
}

}  // namespace streamops
