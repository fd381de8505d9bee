// Interfaces between the C-ABI layer (api.cu) and the kernel families (one .cu file each).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace streamops {

enum : int { OP_COPY = 0, OP_SCALE = 1, OP_ADD = 2, OP_TRIAD = 3, OP_DOT = 4, OP_COUNT = 5 };
enum : int { DT_F32 = 0, DT_F64 = 1 };

constexpr int kMaxThreads = 512;       // __launch_bounds__ of every vector kernel
constexpr int kMaxDotBlocks = 16384;   // partial sums per Dot workspace slot
constexpr int kDotLiveSlots = 24;      // Dot calls on different streams that may be in flight per device
constexpr int kDotCaptureSlots = 8;    // slots set aside for Dot calls recorded into CUDA graphs
constexpr int kDotSlots = kDotLiveSlots + kDotCaptureSlots;

// Resolved launch shape for the register-vector kernels.
struct VecLaunch {
    int vec_bytes;     // 32, 16, or 0 = scalar kernel (pointers not 16-byte aligned)
    int unroll;        // 1, 2, 4
    int policy;        // 0..kNumPolicies-1
    int threads;
    unsigned grid;
    int contiguous;
    int reverse;       // 1 = walk the tiles from the high addresses down
    int pdl;           // 1 = launch with programmatic stream serialization
    int pipeline;      // Dot: 1 = rolling-slot kernel (unroll = slots per thread)
    size_t hot_tiles;  // policies 7, 8: tiles at the start of the traversal whose stores are evict-first
};

// Resolved launch shape for the bulk-copy (TMA) pipeline kernels.
struct BulkLaunch {
    int threads;       // consumer threads (one extra producer warp is added by the launcher)
    unsigned grid;
    int chunk_bytes;
    int stages;
    unsigned wait_limit;   // mbarrier.try_wait attempts before a pipeline wait gives up
};

// Launch helper. With `pdl` the kernel is launched with programmatic stream serialization: its
// blocks may become resident while the previous kernel in the stream is still draining, and
// wait at grid_dependency_wait() until that kernel has completed and its writes are visible.
// That hides the launch latency and block-scheduling ramp between dependent kernels.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                                 cudaStream_t stream, bool pdl, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

#ifdef __CUDACC__
// First statements of every kernel that may be launched with `pdl`: let the next kernel in the
// stream start launching, then wait for the previous one (both are no-ops in a plain launch).
__device__ __forceinline__ void grid_dependency_sync() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

// Per-slot Dot scratch: partial sums written by pass 1, the arrival ticket of the single-launch
// variant, and (shared) the device error flag.
struct DotScratch {
    double *partials;              // kMaxDotBlocks doubles
    // One 64-bit word per slot. Low half: the arrival ticket, zero between calls (blocks add to it
    // through a 32-bit pointer to the word's first four bytes). High half: the sequence number of the
    // last Dot that FINISHED on the slot. The block that finishes a Dot writes the whole word with one
    // store -- (seq << 32) | 0 -- after its last read of the partial sums, which re-arms the ticket and
    // tells the host, when it needs to know, that the slot is free.
    unsigned long long *ticket;
    unsigned seq;                  // this call's sequence number on its slot (0 for slots used by graphs)
};

// api.cu: bookkeeping shared by the entry points that live in other files
int note_cuda_error(cudaError_t e);      // records e, returns STREAMOPS_ERR_CUDA
void note_launches(int n);              // adds to streamops_launch_count

// elementwise.cu
cudaError_t launch_elementwise(int op, int dtype, const VecLaunch &cfg, const void *x, const void *y,
                               void *out, double scalar, size_t n, cudaStream_t stream);
// dot.cu
// `wide`: out is a double that receives the unrounded total, whatever the element type
cudaError_t launch_dot(int dtype, const VecLaunch &cfg, bool two_pass, bool wide, const void *x, const void *y,
                       void *out, size_t n, const DotScratch &scratch, cudaStream_t stream,
                       int *launches);
// the default double-precision Dot with three time stamps per block (see stream_dot_timeline_f64)
cudaError_t launch_dot_timeline(const VecLaunch &cfg, const double *x, const double *y, double *out, size_t n,
                                const DotScratch &scratch, unsigned long long *stamps, cudaStream_t stream);
// dot_comp.cu: Dot with (sum, error) pairs throughout; one launch; cfg.grid <= kMaxDotBlocks / 2
cudaError_t launch_dot_compensated(int dtype, const VecLaunch &cfg, const void *x, const void *y, void *out, size_t n,
                                   const DotScratch &scratch, cudaStream_t stream);
// out[0] = (T)(((p[0] + p[1]) + p[2]) + ...), one thread, index order
cudaError_t launch_fold(int dtype, const double *partials, size_t count, void *out, cudaStream_t stream);
// bulk.cu
cudaError_t launch_bulk(int op, int dtype, const BulkLaunch &cfg, const void *x, const void *y,
                        void *out, double scalar, size_t n, const DotScratch &scratch,
                        int *error_flag, cudaStream_t stream, int *launches);
size_t bulk_smem_bytes(int op, const BulkLaunch &cfg);

}  // namespace streamops
