// Compensated Dot: the same streaming structure as dot.cu with every accumulator carried as a
// (sum, error) pair, for data whose dot product cancels heavily (Table 1's "Dot" with the
// accuracy of a sum done in about twice the working precision).
//
// Per element: the product is split exactly into p + e (p = RN(x*y), e = fma(x, y, -p); for float
// inputs widened to double p is already exact), p is added to the running sum with an error-free
// two-sum, and the two rounding errors go into the running error term. Pairs are merged the same
// way up the fixed thread -> warp -> block -> grid tree, and the final value is RN(sum + error).
// This is the published Dot2 scheme (Ogita, Rump, Oishi) laid out over the GPU's reduction tree;
// its error is about u + n^2 u^2 * cond instead of n u * cond (u = 2^-53). It costs ~10 double-
// precision operations per element instead of one, which the SMs still do faster than HBM
// delivers the operands. Fixed order throughout: repeated calls return identical bits.
#include "internal.cuh"
#include "memops.cuh"
#include "reduce.cuh"

namespace streamops {

namespace {

struct Pair { double s, c; };

__device__ __forceinline__ void two_sum(double a, double b, double &s, double &err) {
    s = __dadd_rn(a, b);
    const double bb = __dsub_rn(s, a);
    err = __dadd_rn(__dsub_rn(a, __dsub_rn(s, bb)), __dsub_rn(b, bb));
}

template <typename T>
__device__ __forceinline__ void add_product(Pair &acc, T xv, T yv) {
    const double x = widen<T>(xv), y = widen<T>(yv);
    const double p = __dmul_rn(x, y);
    double t;
    two_sum(acc.s, p, acc.s, t);
    if constexpr (sizeof(T) == 8) t = __dadd_rn(t, fma(x, y, -p));   // the product's own rounding error
    acc.c = __dadd_rn(acc.c, t);
}

__device__ __forceinline__ Pair merge(const Pair &a, const Pair &b) {
    Pair r;
    double t;
    two_sum(a.s, b.s, r.s, t);
    r.c = __dadd_rn(__dadd_rn(a.c, b.c), t);
    return r;
}

__device__ __forceinline__ Pair warp_merge(Pair v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Pair o;
        o.s = __shfl_xor_sync(0xffffffffu, v.s, off);
        o.c = __shfl_xor_sync(0xffffffffu, v.c, off);
        // both lanes of a pair must compute the same bits: order the operands by lane
        v = ((threadIdx.x & off) == 0) ? merge(v, o) : merge(o, v);
    }
    return v;
}

// Merge over the block; valid in thread 0.
__device__ __forceinline__ Pair block_merge(Pair v, Pair *warp_part) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nwarps = (blockDim.x + 31) >> 5;
    v = warp_merge(v);
    if (lane == 0) warp_part[warp] = v;
    __syncthreads();
    Pair r{0.0, 0.0};
    if (warp == 0) {
        if (lane < nwarps) r = warp_part[lane];
        r = warp_merge(r);
    }
    return r;
}

template <typename T, int U>
__global__ void __launch_bounds__(kMaxThreads, 2)
dot_comp_kernel(const T *x, const T *y, size_t n, double *partials, unsigned long long *ticket, T *out, int vectorised,
                unsigned seq) {
    constexpr int EPV = 32 / (int)sizeof(T);
    __shared__ Pair warp_part[32];
    __shared__ bool is_last;
    grid_dependency_sync();
    Pair acc[U];
#pragma unroll
    for (int u = 0; u < U; ++u) acc[u] = Pair{0.0, 0.0};

    if (vectorised) {
        const char *xb = reinterpret_cast<const char *>(x);
        const char *yb = reinterpret_cast<const char *>(y);
        const uint64_t l2pol = make_evict_first_policy();
        const size_t nvec = n / EPV;
        const size_t tile_vecs = (size_t)blockDim.x * U;
        const size_t ntiles = nvec / tile_vecs;
        for (size_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
            const size_t v0 = tile * tile_vecs + threadIdx.x;
            Vec<32> xv[U], yv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) ldg<4>(xv[u], xb + (v0 + (size_t)u * blockDim.x) * 32, l2pol);
#pragma unroll
            for (int u = 0; u < U; ++u) ldg<4>(yv[u], yb + (v0 + (size_t)u * blockDim.x) * 32, l2pol);
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
                for (int e = 0; e < EPV; ++e)
                    add_product<T>(acc[u], Lanes<T>::get(xv[u].w, e), Lanes<T>::get(yv[u].w, e));
            }
        }
        if (blockIdx.x == (unsigned)(ntiles % gridDim.x)) {      // ragged end, one block
            for (size_t i = ntiles * tile_vecs * EPV + threadIdx.x; i < n; i += blockDim.x)
                add_product<T>(acc[0], x[i], y[i]);
        }
    } else {
        const size_t stride = (size_t)gridDim.x * blockDim.x;
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
            add_product<T>(acc[0], x[i], y[i]);
    }
    Pair t = acc[0];
#pragma unroll
    for (int u = 1; u < U; ++u) t = merge(t, acc[u]);
    const Pair b = block_merge(t, warp_part);

    if (threadIdx.x == 0) {
        partials[2 * blockIdx.x] = b.s;
        partials[2 * blockIdx.x + 1] = b.c;
        is_last = arrive(ticket) == gridDim.x - 1;                // releases the pair, acquires the others'
    }
    __syncthreads();
    if (is_last) {                                                // fixed-order merge of all blocks' pairs
        Pair a{0.0, 0.0};
        for (unsigned k = threadIdx.x; k < gridDim.x; k += blockDim.x)
            a = merge(a, Pair{__ldcg(partials + 2 * k), __ldcg(partials + 2 * k + 1)});
        __syncthreads();                                          // warp_part is reused
        const Pair total = block_merge(a, warp_part);
        if (threadIdx.x == 0) {
            out[0] = (T)__dadd_rn(total.s, total.c);
            rearm(ticket, seq);
        }
    }
}

template <typename T>
cudaError_t launch_t(const VecLaunch &c, const T *x, const T *y, T *out, size_t n, const DotScratch &s, cudaStream_t st) {
    const int vec = c.vec_bytes == 32;
    switch (vec ? c.unroll : 1) {
        case 1: return launch_kernel(dot_comp_kernel<T, 1>, c.grid, c.threads, 0, st, c.pdl != 0, x, y, n, s.partials, s.ticket, out, vec, s.seq);
        case 2: return launch_kernel(dot_comp_kernel<T, 2>, c.grid, c.threads, 0, st, c.pdl != 0, x, y, n, s.partials, s.ticket, out, vec, s.seq);
        case 4: return launch_kernel(dot_comp_kernel<T, 4>, c.grid, c.threads, 0, st, c.pdl != 0, x, y, n, s.partials, s.ticket, out, vec, s.seq);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_dot_compensated(int dtype, const VecLaunch &cfg, const void *x, const void *y, void *out, size_t n,
                                   const DotScratch &scratch, cudaStream_t stream) {
    if (2 * (size_t)cfg.grid > (size_t)kMaxDotBlocks) return cudaErrorInvalidValue;   // two doubles per block
    if (dtype == DT_F64) return launch_t<double>(cfg, (const double *)x, (const double *)y, (double *)out, n, scratch, stream);
    return launch_t<float>(cfg, (const float *)x, (const float *)y, (float *)out, n, scratch, stream);
}

}  // namespace streamops
