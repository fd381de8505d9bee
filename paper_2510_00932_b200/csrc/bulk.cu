// Bulk-copy (TMA) pipeline kernels: the same five operations, with global->shared traffic moved
// by cp.async.bulk and tracked by mbarriers instead of by per-thread vector loads.
//
// Each array is cut into chunks of `chunk_bytes` (the last one shorter, a multiple of 16 bytes;
// elements past it -- fewer than 16 bytes -- are handled by plain loads). Chunk k belongs to
// CTA k mod G. Every CTA owns a ring of S stages in shared memory, each with a "full" mbarrier
// (armed with the byte count of the copies landing in it) and an "empty" mbarrier (released by
// whoever has finished with the stage). One elected thread of the producer warp keeps up to S
// chunks per input array in flight -- far more bytes per SM than registers could hold -- with no
// cluster and no multicast.
//
//   Copy:                    a second elected thread forwards each landed stage with a bulk
//                            shared->global store and releases the stage once the store has
//                            finished reading it. Two threads move all the data.
//   Mul / Add / Triad / Dot: consumer warps read the landed stage from shared memory in
//                            16-byte pieces, apply the same rounded arithmetic as the register
//                            kernels and store the result with 16-byte st.global (Dot: fold it
//                            into per-thread double accumulators, then the shared fixed-order
//                            reduction).
//
// Every wait on an mbarrier is a bounded loop around mbarrier.try_wait (`wait_limit` attempts, a
// kernel argument: 2^22 by default, lowered by streamops_set_wait_limit to exercise this path). A
// wait that runs out writes a code to the device error flag and tells the rest of the CTA to stop;
// the loading thread always waits (bounded) for the copies it has in flight before it returns;
// the host reports STREAMOPS_ERR_TIMEOUT. The output of such a launch is incomplete.
#include "internal.cuh"
#include "memops.cuh"
#include "reduce.cuh"

namespace streamops {

namespace {

constexpr unsigned kDrainLimit = 1u << 22;  // try_wait attempts granted to copies already in flight
constexpr int kMaxStages = 8;

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                 :: "r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait of at most `limit` attempts; false = gave up (or another thread of the CTA already did).
// The first attempt is a probe that never blocks (test_wait); each later one (try_wait) may suspend
// the thread for a hardware-defined time before it reports "not yet". A limit of 1 therefore gives up
// at once unless the phase has already completed.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, unsigned parity, volatile int *stop, unsigned limit) {
    if (mbar_test_wait(bar, parity)) return true;
    for (unsigned i = 1; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && *stop) return false;
    }
    return false;
}
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src_gmem, unsigned bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_addr(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst_gmem, const void *src_smem, unsigned bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(dst_gmem), "r"(smem_addr(src_smem)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" :: "n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void lds16(Vec<16> &v, const void *p) {
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "r"(smem_addr(p)));
}

// Chunk geometry shared by all kernels: `bulk_bytes` (a multiple of 16) is the part moved by
// bulk copies, in `nchunks` chunks of `chunk` bytes, the last possibly shorter.
struct Chunks {
    size_t bulk_bytes, nchunks;
    unsigned chunk;
    __device__ __forceinline__ unsigned size_of(size_t k) const {
        const size_t off = k * chunk;
        return (unsigned)(bulk_bytes - off < chunk ? bulk_bytes - off : chunk);
    }
};
__device__ __forceinline__ Chunks make_chunks(size_t total_bytes, unsigned chunk) {
    Chunks c;
    c.bulk_bytes = total_bytes & ~(size_t)15;
    c.chunk = chunk;
    c.nchunks = (c.bulk_bytes + chunk - 1) / chunk;
    return c;
}

struct Ring {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    int stop;
};

// Last act of every loading thread, whether its loop ended normally or a wait gave up: wait
// (bounded, with the full fixed limit whatever limit the pipeline's own waits run under) until
// the copies it issued last have landed, so that no copy is still writing into this CTA's shared
// memory when the CTA exits. Each of those copies was armed on its stage's "full" barrier, and a
// completed phase stays completed, so this returns at once when the data is already there.
__device__ __forceinline__ void drain_loads(Ring *ring, int stages, size_t issued) {
    int dummy = 0;
    const size_t first = issued > (size_t)stages ? issued - stages : 0;
    for (size_t it = first; it < issued; ++it)
        mbar_wait(&ring->full[it % stages], (unsigned)((it / stages) & 1), &dummy, kDrainLimit);
}

__device__ __forceinline__ void flag_timeout(Ring *ring, int *error_flag, int code) {
    ring->stop = 1;
    atomicExch(error_flag, code);
}

// ------------------------------------------------------------------------------------ Copy
// 64 threads: warp 0 lane 0 loads, warp 1 lane 0 stores; the other lanes only move the tail.
__global__ void __launch_bounds__(64)
bulk_copy_kernel(const char *x, char *out, size_t total_bytes, unsigned chunk, int stages, int *error_flag,
                 unsigned wait_limit) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ Ring ring;
    const Chunks ck = make_chunks(total_bytes, chunk);
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&ring.full[s], 1); mbar_init(&ring.empty[s], 1); }
        ring.stop = 0;
        mbar_init_fence();
    }
    __syncthreads();

    if (threadIdx.x == 0) {                                   // loader
        size_t it = 0;
        for (size_t k = blockIdx.x; k < ck.nchunks; k += gridDim.x, ++it) {
            const int s = (int)(it % stages);
            const unsigned ph = (unsigned)((it / stages) & 1);
            if (!mbar_wait(&ring.empty[s], ph ^ 1u, &ring.stop, wait_limit)) { flag_timeout(&ring, error_flag, 1); break; }
            const unsigned bytes = ck.size_of(k);
            mbar_arrive_expect_tx(&ring.full[s], bytes);
            bulk_load(smem + (size_t)s * chunk, x + k * (size_t)chunk, bytes, &ring.full[s]);
        }
        drain_loads(&ring, stages, it);
    } else if (threadIdx.x == 32) {                           // storer
        size_t it = 0;
        bool ok = true;
        for (size_t k = blockIdx.x; k < ck.nchunks; k += gridDim.x, ++it) {
            const int s = (int)(it % stages);
            const unsigned ph = (unsigned)((it / stages) & 1);
            if (!mbar_wait(&ring.full[s], ph, &ring.stop, wait_limit)) { flag_timeout(&ring, error_flag, 2); ok = false; break; }
            bulk_store(out + k * (size_t)chunk, smem + (size_t)s * chunk, ck.size_of(k));
            bulk_commit();
            if (it > 0) {                                     // the previous store has left its stage
                bulk_wait_read<1>();
                mbar_arrive(&ring.empty[(it - 1) % stages]);
            }
        }
        bulk_wait_read<0>();
        if (ok && it > 0) mbar_arrive(&ring.empty[(it - 1) % stages]);
        bulk_wait_all();
    }
    // bytes past the last 16-byte boundary (at most 15), by block 0
    if (blockIdx.x == 0) {
        const size_t i = ck.bulk_bytes + threadIdx.x;
        if (i < total_bytes) out[i] = x[i];
    }
}

// ------------------------------------------------------------------- Mul / Add / Triad / Dot
template <typename T> __device__ __forceinline__ T mul_rn(T a, T b);
template <> __device__ __forceinline__ double mul_rn<double>(double a, double b) { return __dmul_rn(a, b); }
template <> __device__ __forceinline__ float mul_rn<float>(float a, float b) { return __fmul_rn(a, b); }
template <typename T> __device__ __forceinline__ T add_rn(T a, T b);
template <> __device__ __forceinline__ double add_rn<double>(double a, double b) { return __dadd_rn(a, b); }
template <> __device__ __forceinline__ float add_rn<float>(float a, float b) { return __fadd_rn(a, b); }

template <typename T, int OP>
__device__ __forceinline__ T apply(T x, T y, T s) {
    if constexpr (OP == OP_SCALE) return mul_rn<T>(s, x);
    else if constexpr (OP == OP_ADD) return add_rn<T>(x, y);
    else return add_rn<T>(x, mul_rn<T>(s, y));                // Triad: two roundings
}

// blockDim.x = consumers + 32; the last warp is the producer. Consumers take 16-byte pieces
// t, t + C, ... of each landed chunk. DOT folds into `acc` instead of storing.
template <typename T, int OP, bool SINGLE_LAUNCH>
__global__ void __launch_bounds__(kMaxThreads + 32)
bulk_compute_kernel(const T *x, const T *y, T *out, T s, size_t n, unsigned chunk, int stages,
                    double *partials, unsigned long long *ticket, int *error_flag, unsigned wait_limit, unsigned seq) {
    constexpr bool USES_Y = (OP != OP_SCALE);
    constexpr int EPV = 16 / (int)sizeof(T);
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ Ring ring;
    __shared__ double warp_part[32];
    __shared__ bool is_last;
    const int consumers = (int)blockDim.x - 32;
    const int consumer_warps = consumers >> 5;
    const Chunks ck = make_chunks(n * sizeof(T), chunk);
    const size_t stage_bytes = (size_t)chunk * (USES_Y ? 2 : 1);
    const char *xb = reinterpret_cast<const char *>(x);
    const char *yb = reinterpret_cast<const char *>(y);
    char *ob = reinterpret_cast<char *>(out);

    if (threadIdx.x == 0) {
        for (int st = 0; st < stages; ++st) { mbar_init(&ring.full[st], 1); mbar_init(&ring.empty[st], consumer_warps); }
        ring.stop = 0;
        mbar_init_fence();
    }
    __syncthreads();

    double acc = 0.0;
    if ((int)threadIdx.x >= consumers) {
        if ((int)threadIdx.x == consumers) {                  // producer: one elected thread
            size_t it = 0;
            for (size_t k = blockIdx.x; k < ck.nchunks; k += gridDim.x, ++it) {
                const int st = (int)(it % stages);
                const unsigned ph = (unsigned)((it / stages) & 1);
                if (!mbar_wait(&ring.empty[st], ph ^ 1u, &ring.stop, wait_limit)) { flag_timeout(&ring, error_flag, 3); break; }
                const unsigned bytes = ck.size_of(k);
                unsigned char *stage = smem + (size_t)st * stage_bytes;
                mbar_arrive_expect_tx(&ring.full[st], USES_Y ? 2 * bytes : bytes);
                bulk_load(stage, xb + k * (size_t)chunk, bytes, &ring.full[st]);
                if constexpr (USES_Y) bulk_load(stage + chunk, yb + k * (size_t)chunk, bytes, &ring.full[st]);
            }
            drain_loads(&ring, stages, it);
        }
    } else {
        size_t it = 0;
        for (size_t k = blockIdx.x; k < ck.nchunks; k += gridDim.x, ++it) {
            const int st = (int)(it % stages);
            const unsigned ph = (unsigned)((it / stages) & 1);
            if (!mbar_wait(&ring.full[st], ph, &ring.stop, wait_limit)) { flag_timeout(&ring, error_flag, 4); break; }
            const unsigned bytes = ck.size_of(k);
            const unsigned char *stage = smem + (size_t)st * stage_bytes;
            char *dst = ob + k * (size_t)chunk;
            for (unsigned off = threadIdx.x * 16u; off < bytes; off += (unsigned)consumers * 16u) {
                Vec<16> xv, yv;
                lds16(xv, stage + off);
                if constexpr (USES_Y) lds16(yv, stage + chunk + off);
                if constexpr (OP == OP_DOT) {
#pragma unroll
                    for (int e = 0; e < EPV; ++e)
                        acc = fma(widen<T>(Lanes<T>::get(xv.w, e)), widen<T>(Lanes<T>::get(yv.w, e)), acc);
                } else {
#pragma unroll
                    for (int e = 0; e < EPV; ++e)
                        Lanes<T>::set(xv.w, e, apply<T, OP>(Lanes<T>::get(xv.w, e), Lanes<T>::get(yv.w, e), s));
                    stg<2>(dst + off, xv, 0);
                }
            }
            __syncwarp();
            if ((threadIdx.x & 31) == 0) mbar_arrive(&ring.empty[st]);
        }
        // elements past the last 16-byte boundary (fewer than EPV), by block 0
        if (blockIdx.x == 0) {
            const size_t i = ck.bulk_bytes / sizeof(T) + threadIdx.x;
            if (i < n) {
                if constexpr (OP == OP_DOT) acc = fma(widen<T>(x[i]), widen<T>(y[i]), acc);
                else out[i] = apply<T, OP>(x[i], USES_Y ? y[i] : T(0), s);
            }
        }
    }
    if constexpr (OP == OP_DOT) {
        const double bsum = block_sum(acc, warp_part);
        publish_partial<T, SINGLE_LAUNCH>(bsum, partials, ticket, out, warp_part, &is_last, seq);
    }
}

template <typename K>
cudaError_t allow_smem(K kernel, size_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

template <typename T, int OP>
cudaError_t launch_compute(const BulkLaunch &c, const T *x, const T *y, T *out, double scalar, size_t n,
                           const DotScratch &sc, int *error_flag, cudaStream_t st) {
    const size_t smem = bulk_smem_bytes(OP, c);
    auto kernel = bulk_compute_kernel<T, OP, true>;
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return e;
    kernel<<<c.grid, c.threads + 32, smem, st>>>(x, y, out, (T)scalar, n, (unsigned)c.chunk_bytes, c.stages,
                                                 sc.partials, sc.ticket, error_flag, c.wait_limit, sc.seq);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_bulk_t(int op, const BulkLaunch &c, const T *x, const T *y, T *out, double scalar, size_t n,
                          const DotScratch &sc, int *error_flag, cudaStream_t st) {
    switch (op) {
        case OP_SCALE: return launch_compute<T, OP_SCALE>(c, x, y, out, scalar, n, sc, error_flag, st);
        case OP_ADD:   return launch_compute<T, OP_ADD>(c, x, y, out, scalar, n, sc, error_flag, st);
        case OP_TRIAD: return launch_compute<T, OP_TRIAD>(c, x, y, out, scalar, n, sc, error_flag, st);
        case OP_DOT:
            if (c.grid > (unsigned)kMaxDotBlocks) return cudaErrorInvalidValue;
            return launch_compute<T, OP_DOT>(c, x, y, out, scalar, n, sc, error_flag, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

size_t bulk_smem_bytes(int op, const BulkLaunch &c) {
    const size_t arrays = (op == OP_COPY || op == OP_SCALE) ? 1 : 2;
    return (size_t)c.stages * (size_t)c.chunk_bytes * arrays;
}

cudaError_t launch_bulk(int op, int dtype, const BulkLaunch &c, const void *x, const void *y, void *out,
                        double scalar, size_t n, const DotScratch &scratch, int *error_flag,
                        cudaStream_t stream, int *launches) {
    *launches = 1;
    if (c.stages < 2 || c.stages > kMaxStages || c.chunk_bytes < 16 || (c.chunk_bytes & 15))
        return cudaErrorInvalidValue;
    if (op == OP_COPY) {
        const size_t smem = bulk_smem_bytes(op, c);
        cudaError_t e = allow_smem(bulk_copy_kernel, smem);
        if (e != cudaSuccess) return e;
        const size_t bytes = n * (dtype == DT_F64 ? 8 : 4);
        bulk_copy_kernel<<<c.grid, 64, smem, stream>>>((const char *)x, (char *)out, bytes,
                                                       (unsigned)c.chunk_bytes, c.stages, error_flag, c.wait_limit);
        return cudaGetLastError();
    }
    if (dtype == DT_F64)
        return launch_bulk_t<double>(op, c, (const double *)x, (const double *)y, (double *)out, scalar, n,
                                     scratch, error_flag, stream);
    return launch_bulk_t<float>(op, c, (const float *)x, (const float *)y, (float *)out, scalar, n,
                                scratch, error_flag, stream);
}

}  // namespace streamops
