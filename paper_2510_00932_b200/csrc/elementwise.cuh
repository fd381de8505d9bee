// Register-vector kernels for Copy, Mul (scale), Add and Triad (Table 1 of the paper).
//
// Work is cut into tiles of blockDim.x * U vectors (a vector is 16 or 32 bytes). Inside a tile
// thread t owns vectors t, t + blockDim.x, ..., so that each warp-wide access covers one
// contiguous 512- or 1024-byte span. A thread issues all of a tile's loads (U per input array)
// before the first arithmetic instruction: U * VB bytes per array per thread are in flight,
// which is what hides HBM latency. Blocks walk the tiles either interleaved (tile b, b + G,
// ...) or as one contiguous range per block, from the low addresses up or -- "reverse" -- from the
// high addresses down (a kernel that consumes what the previous kernel just wrote finds the most
// recently written lines still in L2 if it starts where the producer stopped). The ragged end -- vectors past the last full tile,
// then elements past the last full vector -- is handled by one block with bounds checks, using
// the same arithmetic.
//
// Arithmetic uses the explicit round-to-nearest intrinsics (__dmul_rn, __dadd_rn, __fmul_rn,
// __fadd_rn), which the compiler never contracts into a fused multiply-add.
#pragma once
#include "indexcheck.cuh"
#include "internal.cuh"
#include "memops.cuh"

namespace streamops {

template <typename T> __device__ __forceinline__ T mul_rn(T a, T b);
template <> __device__ __forceinline__ double mul_rn<double>(double a, double b) { return __dmul_rn(a, b); }
template <> __device__ __forceinline__ float mul_rn<float>(float a, float b) { return __fmul_rn(a, b); }
template <typename T> __device__ __forceinline__ T add_rn(T a, T b);
template <> __device__ __forceinline__ double add_rn<double>(double a, double b) { return __dadd_rn(a, b); }
template <> __device__ __forceinline__ float add_rn<float>(float a, float b) { return __fadd_rn(a, b); }

// One element of op OP. Copy never reaches here (it moves raw words).
template <typename T, int OP>
__device__ __forceinline__ T apply(T x, T y, T s) {
    if constexpr (OP == OP_SCALE) return mul_rn<T>(s, x);
    else if constexpr (OP == OP_ADD) return add_rn<T>(x, y);
    else return add_rn<T>(x, mul_rn<T>(s, y));   // Triad: rounded product, then rounded sum
}

template <int OP> constexpr bool kUsesY = (OP == OP_ADD || OP == OP_TRIAD);

template <typename T, int OP, int VB>
__device__ __forceinline__ void apply_vec(Vec<VB> &xv, const Vec<VB> &yv, T s) {
    if constexpr (OP != OP_COPY) {
        constexpr int EPV = VB / (int)sizeof(T);
#pragma unroll
        for (int e = 0; e < EPV; ++e)
            Lanes<T>::set(xv.w, e, apply<T, OP>(Lanes<T>::get(xv.w, e), Lanes<T>::get(yv.w, e), s));
    }
}

template <typename T, int OP, int VB, int U, int POL>
__global__ void __launch_bounds__(kMaxThreads)
ew_vec_kernel(const T *x, const T *y, T *out, T s, size_t n, int contiguous, int reverse, size_t hot_tiles) {
    constexpr int EPV = VB / (int)sizeof(T);
    grid_dependency_sync();
    const char *xb = reinterpret_cast<const char *>(x);
    const char *yb = reinterpret_cast<const char *>(y);
    char *ob = reinterpret_cast<char *>(out);
    const L2Policies l2 = make_l2_policies<POL>();

    const size_t nvec = n / EPV;
    const size_t tile_vecs = (size_t)blockDim.x * U;
    const size_t ntiles = nvec / tile_vecs;          // full tiles only
    const size_t nbytes = n * sizeof(T);             // what index_ok checks against (checking builds only)
    size_t tile, end, step;
    if (contiguous) {
        const size_t per = (ntiles + gridDim.x - 1) / gridDim.x;
        tile = (size_t)blockIdx.x * per;
        end = tile + per < ntiles ? tile + per : ntiles;
        step = 1;
    } else {
        tile = blockIdx.x; end = ntiles; step = gridDim.x;
    }
    for (; tile < end; tile += step) {
        const size_t v0 = (reverse ? ntiles - 1 - tile : tile) * tile_vecs + threadIdx.x;
        // two-phase stores: the first hot_tiles tiles of the traversal leave L2 first
        const uint64_t stpol = (POL == 8 && tile >= hot_tiles) ? l2.st_late : l2.st;
        Vec<VB> xv[U], yv[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (index_ok((v0 + (size_t)u * blockDim.x) * VB, VB, nbytes, W_EW_LOAD_X))
                ldg<POL>(xv[u], xb + (v0 + (size_t)u * blockDim.x) * VB, l2.ld);
        if constexpr (kUsesY<OP>) {
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (index_ok((v0 + (size_t)u * blockDim.x) * VB, VB, nbytes, W_EW_LOAD_Y))
                    ldg<POL>(yv[u], yb + (v0 + (size_t)u * blockDim.x) * VB, l2.ld);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) apply_vec<T, OP, VB>(xv[u], yv[u], s);
        if (POL == 7 && tile >= hot_tiles) {       // second phase of policy 7: plain stores (uniform per tile)
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (index_ok((v0 + (size_t)u * blockDim.x) * VB, VB, nbytes, W_EW_STORE))
                    stg<0>(ob + (v0 + (size_t)u * blockDim.x) * VB, xv[u], 0);
        } else {
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (index_ok((v0 + (size_t)u * blockDim.x) * VB, VB, nbytes, W_EW_STORE))
                    stg<POL>(ob + (v0 + (size_t)u * blockDim.x) * VB, xv[u], stpol);
        }
    }
    // ragged end, by the block that is next in line for a tile
    if (blockIdx.x == (unsigned)(ntiles % gridDim.x)) {
        for (size_t v = ntiles * tile_vecs + threadIdx.x; v < nvec; v += blockDim.x) {
            Vec<VB> xv, yv;
            if (!index_ok(v * VB, VB, nbytes, W_EW_TAIL)) continue;
            ldg<0>(xv, xb + v * VB, 0);
            if constexpr (kUsesY<OP>) ldg<0>(yv, yb + v * VB, 0);
            apply_vec<T, OP, VB>(xv, yv, s);
            stg<0>(ob + v * VB, xv, 0);
        }
        const size_t i = nvec * EPV + threadIdx.x;   // fewer than EPV elements remain
        if (i < n && index_ok(i * sizeof(T), sizeof(T), nbytes, W_EW_TAIL)) {
            if constexpr (OP == OP_COPY) out[i] = x[i];
            else out[i] = apply<T, OP>(x[i], kUsesY<OP> ? y[i] : T(0), s);
        }
    }
}

// Scalar kernel: any element-aligned pointers. Same arithmetic, one element per access.
template <typename T, int OP>
__global__ void __launch_bounds__(kMaxThreads)
ew_scalar_kernel(const T *x, const T *y, T *out, T s, size_t n) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        if constexpr (OP == OP_COPY) out[i] = x[i];
        else out[i] = apply<T, OP>(x[i], kUsesY<OP> ? y[i] : T(0), s);
    }
}

// Copy moves words, so both element types share the unsigned-word instantiation.
template <typename T> struct WordOf;
template <> struct WordOf<double> { using type = unsigned long long; };
template <> struct WordOf<float> { using type = unsigned int; };

template <typename T, int OP, int VB, int U>
cudaError_t launch_vec_pol(const VecLaunch &c, const T *x, const T *y, T *out, T s, size_t n, cudaStream_t st) {
    switch (c.policy) {
#define STREAMOPS_CASE(P) case P: return launch_kernel(ew_vec_kernel<T, OP, VB, U, P>, c.grid, c.threads, 0, st, c.pdl != 0, x, y, out, s, n, c.contiguous, c.reverse, c.hot_tiles);
        STREAMOPS_CASE(0) STREAMOPS_CASE(1) STREAMOPS_CASE(2) STREAMOPS_CASE(3) STREAMOPS_CASE(4) STREAMOPS_CASE(5) STREAMOPS_CASE(6) STREAMOPS_CASE(7) STREAMOPS_CASE(8)
#undef STREAMOPS_CASE
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

template <typename T, int OP, int VB>
cudaError_t launch_vec_unroll(const VecLaunch &c, const T *x, const T *y, T *out, T s, size_t n, cudaStream_t st) {
    switch (c.unroll) {
        case 1: return launch_vec_pol<T, OP, VB, 1>(c, x, y, out, s, n, st);
        case 2: return launch_vec_pol<T, OP, VB, 2>(c, x, y, out, s, n, st);
        case 4: return launch_vec_pol<T, OP, VB, 4>(c, x, y, out, s, n, st);
        default: return cudaErrorInvalidValue;
    }
}

template <typename T, int OP>
cudaError_t launch_op(const VecLaunch &c, const T *x, const T *y, T *out, double scalar, size_t n, cudaStream_t st) {
    const T s = (T)scalar;   // the scalar's single rounding to the element type
    if (c.vec_bytes == 32) return launch_vec_unroll<T, OP, 32>(c, x, y, out, s, n, st);
    if (c.vec_bytes == 16) return launch_vec_unroll<T, OP, 16>(c, x, y, out, s, n, st);
    ew_scalar_kernel<T, OP><<<c.grid, c.threads, 0, st>>>(x, y, out, s, n);
    return cudaGetLastError();
}

#define STREAMOPS_DECLARE_OP(T, OP) \
    extern template cudaError_t launch_op<T, OP>(const VecLaunch &, const T *, const T *, T *, double, size_t, cudaStream_t);
STREAMOPS_DECLARE_OP(unsigned long long, OP_COPY)
STREAMOPS_DECLARE_OP(unsigned int, OP_COPY)
STREAMOPS_DECLARE_OP(double, OP_SCALE) STREAMOPS_DECLARE_OP(float, OP_SCALE)
STREAMOPS_DECLARE_OP(double, OP_ADD)   STREAMOPS_DECLARE_OP(float, OP_ADD)
STREAMOPS_DECLARE_OP(double, OP_TRIAD) STREAMOPS_DECLARE_OP(float, OP_TRIAD)
#undef STREAMOPS_DECLARE_OP

}  // namespace streamops
