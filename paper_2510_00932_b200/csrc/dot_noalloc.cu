// stream_dot_noalloc_f64: a Dot for callers that must not allocate device memory.
//
// Some callers cannot reach cudaMalloc at the moment they need a dot product: code running inside
// a memory pool that owns the whole device, a latency-critical loop that may not take the
// allocator's lock or its implicit synchronisation, a host application whose policy is that
// libraries never allocate. The regular stream_dot_* entry points keep their partial sums in a
// workspace that the library allocates on first use; this one keeps them in a fixed array that is
// part of the library image instead, so the call path contains no cudaMalloc, no cudaFree and no
// allocating library routine at all. The price is a maximum problem size and no concurrency: the
// array is one per device, every call uses it, and it keeps whatever the previous call left there.
//
// Kernel: block b owns elements [b*SPAN, (b+1)*SPAN) and writes partials[b]; the block that draws
// the last ticket folds the partials in index order (same fixed-order folds as the regular Dot,
// so repeated calls return identical bits). SPAN is fixed, so the scratch array's size fixes the
// largest n.
#include <mutex>

#include "../../include/streamops.h"
#include "internal.cuh"
#include "memops.cuh"
#include "reduce.cuh"

namespace {

using namespace streamops;

constexpr int kThreads = 512;
constexpr int kUnroll = 4;                              // 32-byte vectors per thread per array in flight
constexpr size_t kTile = (size_t)kThreads * kUnroll * 4;   // elements per tile (4 doubles per vector)
constexpr size_t kSpan = 8 * kTile;                     // 65,536 elements per block and per partial sum
constexpr int kMaxBlocks = STREAMOPS_DOT_NOALLOC_MAX_N / kSpan;   // 4096 partial sums
constexpr int kTicketSlot = kMaxBlocks;                 // the ticket lives after the partials
constexpr int kScratchDoubles = kMaxBlocks + 32;        // + 256 bytes holding the ticket
static_assert((size_t)kMaxBlocks * kSpan == STREAMOPS_DOT_NOALLOC_MAX_N, "max n is a whole number of spans");

// The scratch itself: 33,024 bytes in the image of every device that loads the library, held
// until the process exits. In HOST code this name is only a handle for cudaGetSymbolAddress; it
// is not a device address and must never be passed to a kernel.
static __device__ __align__(256) double g_dot_noalloc_scratch[kScratchDoubles];

__global__ void __launch_bounds__(kThreads)
dot_noalloc_kernel(const double *x, const double *y, size_t n, double *scratch, double *out, int vectorised) {
    __shared__ double warp_part[32];
    __shared__ bool is_last;
    double *partials = scratch;
    unsigned long long *ticket = reinterpret_cast<unsigned long long *>(scratch + kTicketSlot);

    const size_t begin = (size_t)blockIdx.x * kSpan;
    const size_t len = n - begin < kSpan ? n - begin : kSpan;
    const double *xs = x + begin, *ys = y + begin;
    double acc[kUnroll] = {0.0, 0.0, 0.0, 0.0};
    if (vectorised) {
        const size_t nvec = len / 4;
        const size_t full = nvec / ((size_t)kThreads * kUnroll) * ((size_t)kThreads * kUnroll);
        for (size_t v0 = threadIdx.x; v0 < full; v0 += (size_t)kThreads * kUnroll) {
            Vec<32> xv[kUnroll], yv[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) ldg<0>(xv[u], xs + (v0 + (size_t)u * kThreads) * 4, 0);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) ldg<0>(yv[u], ys + (v0 + (size_t)u * kThreads) * 4, 0);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    acc[u] = fma(Lanes<double>::get(xv[u].w, e), Lanes<double>::get(yv[u].w, e), acc[u]);
        }
        for (size_t v = full + threadIdx.x; v < nvec; v += kThreads) {     // vectors past the last full tile
            Vec<32> xv, yv;
            ldg<0>(xv, xs + v * 4, 0);
            ldg<0>(yv, ys + v * 4, 0);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                acc[0] = fma(Lanes<double>::get(xv.w, e), Lanes<double>::get(yv.w, e), acc[0]);
        }
        const size_t i = nvec * 4 + threadIdx.x;                            // fewer than 4 elements remain
        if (i < len) acc[0] = fma(xs[i], ys[i], acc[0]);
    } else {
        for (size_t i = threadIdx.x; i < len; i += kThreads) acc[0] = fma(xs[i], ys[i], acc[0]);
    }
    const double tsum = ((acc[0] + acc[1]) + acc[2]) + acc[3];
    const double bsum = block_sum(tsum, warp_part);
    publish_partial<double, true>(bsum, partials, ticket, out, warp_part, &is_last, 0u);
}

// Device address of the scratch array, looked up once per device with that device current.
constexpr int kMaxDevices = 64;
double *g_scratch_ptr[kMaxDevices];
std::mutex g_setup_mutex;

cudaError_t scratch_for_current_device(double **ptr) {
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return e;
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[device]) {
        double *p = nullptr;
        e = cudaGetSymbolAddress((void **)&p, g_dot_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[device] = p;
    }
    *ptr = g_scratch_ptr[device];
    return cudaSuccess;
}

bool overlaps(const void *a, size_t abytes, const void *b, size_t bbytes) {
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + bbytes && b0 < a0 + abytes;
}

}  // namespace

extern "C" int stream_dot_noalloc_f64(const double *x, const double *y, double *out, double scalar, size_t n,
                                      streamops_stream_t stream_) {
    (void)scalar;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!out || (n > 0 && (!x || !y))) return STREAMOPS_ERR_NULL;
    if (((uintptr_t)out % 8) || (n > 0 && (((uintptr_t)x % 8) || ((uintptr_t)y % 8)))) return STREAMOPS_ERR_ALIGN;
    if (n > (size_t)STREAMOPS_DOT_NOALLOC_MAX_N) return STREAMOPS_ERR_TOO_LARGE;
    if (n > 0 && (overlaps(x, n * 8, out, 8) || overlaps(y, n * 8, out, 8))) return STREAMOPS_ERR_OVERLAP;
    cudaError_t e;
    if (n == 0) return (e = cudaMemsetAsync(out, 0, sizeof(double), stream)) == cudaSuccess ? STREAMOPS_OK : note_cuda_error(e);

    double *scratch = nullptr;
    if ((e = scratch_for_current_device(&scratch)) != cudaSuccess) return note_cuda_error(e);
    // the array keeps the last call's contents: the ticket must start at zero (an interrupted
    // earlier call could have left it mid-count); the partial sums are all rewritten before use
    if ((e = cudaMemsetAsync(scratch + kTicketSlot, 0, sizeof(unsigned long long), stream)) != cudaSuccess) return note_cuda_error(e);
    const unsigned blocks = (unsigned)((n + kSpan - 1) / kSpan);
    const int vectorised = (((uintptr_t)x | (uintptr_t)y) & 31) == 0;
    dot_noalloc_kernel<<<blocks, kThreads, 0, stream>>>(x, y, n, scratch, out, vectorised);
    if ((e = cudaGetLastError()) != cudaSuccess) return note_cuda_error(e);
    note_launches(1);                      // host-side counters: nothing here allocates
    return STREAMOPS_OK;
}
