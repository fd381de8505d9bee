// The C ABI of libstreamops: argument checks, per-device state, tuning table, dispatch.
// Declarations and the contract of every entry point are in include/streamops.h.
#include <atomic>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/streamops.h"
#include "internal.cuh"

using namespace streamops;

namespace {

constexpr int kMaxDevices = 64;

struct DeviceState {
    bool ready = false;
    int sm_count = 0;
    double *partials = nullptr;        // kDotSlots * kMaxDotBlocks doubles
    unsigned *tickets = nullptr;       // kDotSlots counters, zero between calls
    int *error_flag = nullptr;         // set by a bounded wait that gave up
    std::atomic<unsigned> next_slot{0};
    // the array most recently written by an elementwise kernel on this device and the end of it that
    // was written last (1 = high addresses): where its still-cached lines are. Packed into atomics;
    // a stale or torn reading only costs bandwidth.
    std::atomic<uintptr_t> last_written{0};
    std::atomic<size_t> last_written_bytes{0};
    std::atomic<int> last_written_end_high{0};
    // host-path buffers (streamops_chain_host_*)
    void *chain_buf[3] = {nullptr, nullptr, nullptr};
    void *chain_dot = nullptr;
    double *chain_partials = nullptr;                  // one double per piece
    size_t chain_bytes = 0;
    cudaStream_t chain_streams[3] = {nullptr, nullptr, nullptr};   // upload, kernels, download
    std::vector<cudaEvent_t> chain_events;
};

DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;
std::atomic<int> g_last_cuda_error{0};
std::atomic<unsigned long long> g_launches{0};

// Defaults: the measured best launch shapes on B200 for arrays far larger than L2 (fp64 n = 2^25,
// fp32 n = 2^26). The elementwise kernels run one block per tile: the hardware block scheduler
// then balances the two dies' unequal distance to memory better than a static persistent grid.
// L2 use across consecutive kernels: loads are marked evict-first (read-once data), and a kernel that
// reads the array the previous kernel wrote walks it from the end that kernel wrote last (reverse = 2,
// automatic): in the sequence copy, scale, add, triad, dot that makes scale and triad walk backwards,
// and every kernel starts where its producer stopped and finds the producer's last-written lines
// still in L2. Stores are two-phase: evict-first while the kernel is still reading those inherited lines
// (its own output would otherwise push them out), normal priority for the last 112 MiB it writes,
// which is what it leaves behind for its consumer (measured at fp64 n = 2^25: 337 MB, 16 %, fewer
// DRAM reads per pass of the five kernels than with no reuse; 297 MB with one-phase stores).
// Programmatic dependent launch is on: back-to-back kernels of one stream overlap launch latency
// with the predecessor's tail (measured: 2 us per launch).
streamops_tuning_t default_tuning(int op, int dtype) {
    streamops_tuning_t t;
    t.kind = 0; t.vec_bytes = 32; t.unroll = 2; t.threads = 256; t.blocks_per_sm = 0;
    t.policy = 7; t.contiguous = 0; t.chunk_bytes = 16384; t.stages = 4; t.two_pass = 0; t.reverse = 0; t.pdl = 1; t.keep_mib = 112; t.compensated = 0;
    const bool f64 = dtype == DT_F64;
    switch (op) {
        case OP_COPY:  t.reverse = 2; break;
        case OP_SCALE: t.reverse = 2; break;
        case OP_ADD:   t.threads = 128; t.reverse = 2; break;
        case OP_TRIAD: t.threads = 128; t.reverse = 2; break;
        // Dot, double: persistent grid sized automatically (blocks_per_sm = 0: 2 or 3 per SM, see
        // resolve_vec); float: 2 per SM and two vectors in flight measured best from 16 MiB to 2 GiB
        case OP_DOT:   t.threads = 512; t.policy = 4; t.unroll = f64 ? 4 : 2; t.blocks_per_sm = f64 ? 0 : 2; break;
    }
    return t;
}

streamops_tuning_t g_tuning[OP_COUNT][2];
std::once_flag g_tuning_once;
void init_tuning() {
    for (int op = 0; op < OP_COUNT; ++op)
        for (int dt = 0; dt < 2; ++dt) g_tuning[op][dt] = default_tuning(op, dt);
}
const streamops_tuning_t &tuning(int op, int dtype) {
    std::call_once(g_tuning_once, init_tuning);
    return g_tuning[op][dtype];
}

int cuda_fail(cudaError_t e) {
    g_last_cuda_error.store((int)e);
    return STREAMOPS_ERR_CUDA;
}

int init_device(int device, DeviceState **out) {
    if (device < 0 || device >= kMaxDevices) return STREAMOPS_ERR_ARG;
    DeviceState &d = g_dev[device];
    if (!d.ready) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!d.ready) {
            int prev = 0;
            cudaError_t e = cudaGetDevice(&prev);
            if (e != cudaSuccess) return cuda_fail(e);
            if ((e = cudaSetDevice(device)) != cudaSuccess) return cuda_fail(e);
            int status = STREAMOPS_OK;
            do {
                if ((e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess) { status = cuda_fail(e); break; }
                const size_t pbytes = sizeof(double) * kDotSlots * kMaxDotBlocks;
                if (cudaMalloc(&d.partials, pbytes) != cudaSuccess ||
                    cudaMalloc(&d.tickets, sizeof(unsigned) * kDotSlots) != cudaSuccess ||
                    cudaMalloc(&d.error_flag, sizeof(int)) != cudaSuccess) {
                    (void)cudaGetLastError();
                    status = STREAMOPS_ERR_WORKSPACE; break;
                }
                if ((e = cudaMemset(d.tickets, 0, sizeof(unsigned) * kDotSlots)) != cudaSuccess) { status = cuda_fail(e); break; }
                if ((e = cudaMemset(d.error_flag, 0, sizeof(int))) != cudaSuccess) { status = cuda_fail(e); break; }
            } while (false);
            cudaSetDevice(prev);
            if (status != STREAMOPS_OK) {
                cudaFree(d.partials); cudaFree(d.tickets); cudaFree(d.error_flag);
                d.partials = nullptr; d.tickets = nullptr; d.error_flag = nullptr;
                return status;
            }
            d.ready = true;
        }
    }
    *out = &d;
    return STREAMOPS_OK;
}

int current_device_state(DeviceState **out) {
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(e);
    return init_device(device, out);
}

bool ranges_overlap(const void *a, size_t abytes, const void *b, size_t bbytes) {
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + bbytes && b0 < a0 + abytes;
}

// Null / alignment / overlap rules common to the five operations.
int check_args(int op, size_t esize, const void *x, const void *y, const void *out, size_t n, size_t out_esize) {
    const bool uses_y = (op == OP_ADD || op == OP_TRIAD || op == OP_DOT);
    if (!out && (n > 0 || op == OP_DOT)) return STREAMOPS_ERR_NULL;   // Dot writes even for n == 0
    if (n > 0 && (!x || (uses_y && !y))) return STREAMOPS_ERR_NULL;
    if (((uintptr_t)out % out_esize) || (n > 0 && (((uintptr_t)x % esize) || (uses_y && ((uintptr_t)y % esize)))))
        return STREAMOPS_ERR_ALIGN;
    if (n == 0) return STREAMOPS_OK;
    if (n > ((size_t)1 << 48)) return STREAMOPS_ERR_ARG;
    const size_t bytes = n * esize;
    const size_t obytes = (op == OP_DOT) ? out_esize : bytes;
    const void *ins[2] = {x, uses_y ? y : nullptr};
    for (const void *in : ins) {
        if (!in) continue;
        if (op != OP_DOT && in == out) continue;              // exact in-place use is allowed
        if (ranges_overlap(in, bytes, out, obytes)) return STREAMOPS_ERR_OVERLAP;
    }
    return STREAMOPS_OK;
}

unsigned clamp_grid(size_t blocks) {
    if (blocks < 1) return 1;
    return (unsigned)(blocks > 0x7fffffffull ? 0x7fffffffull : blocks);
}

VecLaunch resolve_vec(const streamops_tuning_t &t, const DeviceState &d, int op, size_t esize,
                      const void *x, const void *y, const void *out, size_t n) {
    VecLaunch c;
    uintptr_t bits = (uintptr_t)x | (op == OP_DOT ? 0 : (uintptr_t)out);
    if (op == OP_ADD || op == OP_TRIAD || op == OP_DOT) bits |= (uintptr_t)y;
    c.vec_bytes = t.vec_bytes;
    if (c.vec_bytes == 32 && (bits & 31)) c.vec_bytes = 16;
    if (c.vec_bytes == 16 && (bits & 15)) c.vec_bytes = 0;
    c.unroll = t.unroll;
    c.threads = t.threads;
    c.contiguous = t.contiguous;
    c.reverse = t.reverse == 1;                                  // 2 (automatic) is resolved by the caller
    c.pdl = t.pdl != 0;
    c.policy = t.policy;
    // the read-only data path must not be used on an array the kernel also writes
    if (c.policy == 1 && (out == x || out == y)) c.policy = 0;
    if (op == OP_DOT && c.policy > 6) c.policy = 4;           // Dot stores nothing: the two-phase sets reduce to 4
    const size_t per_tile = (size_t)c.threads * (c.vec_bytes ? (size_t)c.unroll * c.vec_bytes / esize : 1);
    const size_t tiles = (n + per_tile - 1) / per_tile;
    size_t grid = t.blocks_per_sm > 0 ? (size_t)t.blocks_per_sm * d.sm_count : tiles;
    if (op == OP_DOT && t.blocks_per_sm == 0) {
        // automatic persistent grid: a third block per SM (which starts as the first two finish and
        // evens out the tail) pays once every block has several tiles; small arrays do best with two
        const size_t three = (size_t)3 * d.sm_count;
        grid = tiles >= 6 * three ? three : (size_t)2 * d.sm_count;
    }
    if (grid > tiles) grid = tiles;                            // never more blocks than tiles
    if (op == OP_DOT && grid > (size_t)kMaxDotBlocks) grid = kMaxDotBlocks;
    c.grid = clamp_grid(grid);
    const size_t keep_tiles = ((size_t)t.keep_mib << 20) / (per_tile * esize);
    c.hot_tiles = tiles > keep_tiles ? tiles - keep_tiles : 0;
    return c;
}

bool valid_tuning(const streamops_tuning_t &t) {
    if (t.kind != 0 && t.kind != 1) return false;
    if (t.vec_bytes != 16 && t.vec_bytes != 32) return false;
    if (t.unroll != 1 && t.unroll != 2 && t.unroll != 4) return false;
    if (t.threads != 128 && t.threads != 256 && t.threads != 512) return false;
    if (t.blocks_per_sm < 0 || t.blocks_per_sm > 32) return false;
    if (t.policy < 0 || t.policy > 8) return false;
    if (t.keep_mib < 0 || t.keep_mib > 65536) return false;
    if (t.compensated != 0 && t.compensated != 1) return false;
    if (t.chunk_bytes < 1024 || t.chunk_bytes > 65536 || (t.chunk_bytes & 15)) return false;
    if (t.stages < 2 || t.stages > 8) return false;
    if (t.reverse < 0 || t.reverse > 2) return false;
    return true;
}

// `wide` (Dot only): out is one double receiving the unrounded total.
int run_op(int op, int dtype, const void *x, const void *y, void *out, double scalar, size_t n,
           streamops_stream_t stream_, bool wide = false) {
    cudaStream_t stream = (cudaStream_t)stream_;
    const size_t esize = dtype == DT_F64 ? 8 : 4;
    const size_t out_esize = wide ? 8 : esize;
    int status = check_args(op, esize, x, y, out, n, out_esize);
    if (status != STREAMOPS_OK) return status;
    if (n == 0) {
        if (op != OP_DOT) return STREAMOPS_OK;
        cudaError_t e = cudaMemsetAsync(out, 0, out_esize, stream);   // +0 in either format
        return e == cudaSuccess ? STREAMOPS_OK : cuda_fail(e);
    }
    DeviceState *d = nullptr;
    if ((status = current_device_state(&d)) != STREAMOPS_OK) return status;
    const streamops_tuning_t &t = tuning(op, dtype);

    DotScratch scratch{nullptr, nullptr};
    if (op == OP_DOT) {
        const unsigned slot = d->next_slot.fetch_add(1) % kDotSlots;
        scratch.partials = d->partials + (size_t)slot * kMaxDotBlocks;
        scratch.ticket = d->tickets + slot;
    }

    cudaError_t e;
    int launches = 1;
    const bool uses_y = (op == OP_ADD || op == OP_TRIAD || op == OP_DOT);
    uintptr_t bits = (uintptr_t)x | (op == OP_DOT ? 0 : (uintptr_t)out);
    if (uses_y) bits |= (uintptr_t)y;
    if (t.kind == 1 && !(bits & 15) && !wide) {
        BulkLaunch b;
        b.threads = t.threads;
        b.chunk_bytes = t.chunk_bytes;
        b.stages = t.stages;
        const size_t nchunks = (n * esize + b.chunk_bytes - 1) / b.chunk_bytes;
        size_t grid = (size_t)(t.blocks_per_sm > 0 ? t.blocks_per_sm : 1) * d->sm_count;
        if (grid > nchunks) grid = nchunks;
        if (op == OP_DOT && grid > (size_t)kMaxDotBlocks) grid = kMaxDotBlocks;
        b.grid = clamp_grid(grid);
        e = launch_bulk(op, dtype, b, x, y, out, scalar, n, scratch, d->error_flag, stream, &launches);
    } else {
        VecLaunch c = resolve_vec(t, *d, op, esize, x, y, out, n);
        if (op != OP_DOT) {
            if (t.reverse == 2) {
                // automatic direction: if an input is the array the previous elementwise kernel wrote,
                // start at the end that kernel wrote last (its lines are the ones still in L2)
                const uintptr_t w = d->last_written.load();
                const bool consumer = w != 0 && d->last_written_bytes.load() == n * esize &&
                                      (w == (uintptr_t)x || (uses_y && w == (uintptr_t)y));
                c.reverse = consumer && d->last_written_end_high.load() != 0;
            }
            d->last_written.store((uintptr_t)out);
            d->last_written_bytes.store(n * esize);
            d->last_written_end_high.store(c.reverse ? 0 : 1);       // a forward walk finishes at the high end
        }
        if (op == OP_DOT && t.compensated && !wide) {
            VecLaunch cc = c;
            if (cc.vec_bytes != 32) cc.vec_bytes = 0;                    // 32-byte vectors or the scalar loop
            if (cc.grid > (unsigned)kMaxDotBlocks / 2) cc.grid = kMaxDotBlocks / 2;
            e = launch_dot_compensated(dtype, cc, x, y, out, n, scratch, stream);
        } else if (op == OP_DOT) e = launch_dot(dtype, c, t.two_pass != 0, wide, x, y, out, n, scratch, stream, &launches);
        else e = launch_elementwise(op, dtype, c, x, y, out, scalar, n, stream);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    g_launches.fetch_add((unsigned long long)launches);
    return STREAMOPS_OK;
}

// Host-buffer pass, pipelined: the arrays are cut into pieces of g_chain_piece_bytes per array; piece k
// is uploaded on one stream, run through the five kernels on a second (Dot as a double partial sum
// per piece), and downloaded on a third, so that uploads, kernels and downloads of different pieces
// overlap and the two directions of the host link are busy at the same time. The dot product is the
// left-to-right fold of the per-piece partial sums: fixed by n alone, so repeatable bit for bit.
std::atomic<size_t> g_chain_piece_bytes{(size_t)16 << 20};
constexpr size_t kChainMaxPieces = 4096;

template <typename T>
int chain_host(T *a, T *b, T *c, double scalar, size_t n, T *dot_out) {
    constexpr int dtype = sizeof(T) == 8 ? DT_F64 : DT_F32;
    if (!dot_out || (n > 0 && (!a || !b || !c))) return STREAMOPS_ERR_NULL;
    DeviceState *d = nullptr;
    int status = current_device_state(&d);
    if (status != STREAMOPS_OK) return status;
    std::lock_guard<std::mutex> lock(g_mutex);
    cudaError_t e;
    const size_t bytes = n * sizeof(T);
    for (cudaStream_t &st : d->chain_streams)
        if (!st && (e = cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
    if (!d->chain_dot && (cudaMalloc(&d->chain_dot, 8) != cudaSuccess ||
                          cudaMalloc(&d->chain_partials, sizeof(double) * kChainMaxPieces) != cudaSuccess)) {
        (void)cudaGetLastError();
        return STREAMOPS_ERR_WORKSPACE;
    }
    if (bytes > d->chain_bytes) {
        for (void *&p : d->chain_buf) { cudaFree(p); p = nullptr; }
        d->chain_bytes = 0;
        for (void *&p : d->chain_buf)
            if (cudaMalloc(&p, bytes) != cudaSuccess) { (void)cudaGetLastError(); return STREAMOPS_ERR_WORKSPACE; }
        d->chain_bytes = bytes;
    }
    // pieces: whole multiples of 32 bytes, at most kChainMaxPieces of them
    size_t piece = g_chain_piece_bytes.load() / sizeof(T);
    while ((n + piece - 1) / piece > kChainMaxPieces) piece *= 2;
    const size_t pieces = n ? (n + piece - 1) / piece : 0;
    while (d->chain_events.size() < 2 * pieces) {
        cudaEvent_t ev;
        if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        d->chain_events.push_back(ev);
    }
    cudaStream_t up = d->chain_streams[0], run = d->chain_streams[1], down = d->chain_streams[2];
    T *host[3] = {a, b, c};
    T *dev[3] = {(T *)d->chain_buf[0], (T *)d->chain_buf[1], (T *)d->chain_buf[2]};
    T *dd = (T *)d->chain_dot;
    for (size_t k = 0; k < pieces; ++k) {
        const size_t lo = k * piece, len = n - lo < piece ? n - lo : piece;
        cudaEvent_t uploaded = d->chain_events[2 * k], computed = d->chain_events[2 * k + 1];
        for (int i = 0; i < 3; ++i)
            if ((e = cudaMemcpyAsync(dev[i] + lo, host[i] + lo, len * sizeof(T), cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventRecord(uploaded, up)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(run, uploaded, 0)) != cudaSuccess) return cuda_fail(e);
        T *pa = dev[0] + lo, *pb = dev[1] + lo, *pc = dev[2] + lo;
        // c <- a; b <- s*c; c <- a+b; a <- b+s*c; partial dot(a, b)
        if ((status = run_op(OP_COPY, dtype, pa, nullptr, pc, scalar, len, run)) != STREAMOPS_OK) return status;
        if ((status = run_op(OP_SCALE, dtype, pc, nullptr, pb, scalar, len, run)) != STREAMOPS_OK) return status;
        if ((status = run_op(OP_ADD, dtype, pa, pb, pc, scalar, len, run)) != STREAMOPS_OK) return status;
        if ((status = run_op(OP_TRIAD, dtype, pb, pc, pa, scalar, len, run)) != STREAMOPS_OK) return status;
        if ((status = run_op(OP_DOT, dtype, pa, pb, d->chain_partials + k, scalar, len, run, dtype == DT_F32)) != STREAMOPS_OK) return status;
        if ((e = cudaEventRecord(computed, run)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(down, computed, 0)) != cudaSuccess) return cuda_fail(e);
        for (int i = 0; i < 3; ++i)
            if ((e = cudaMemcpyAsync(host[i] + lo, dev[i] + lo, len * sizeof(T), cudaMemcpyDeviceToHost, down)) != cudaSuccess) return cuda_fail(e);
    }
    if ((e = launch_fold(dtype, d->chain_partials, pieces, dd, run)) != cudaSuccess) return cuda_fail(e);
    g_launches.fetch_add(1);
    if ((e = cudaMemcpyAsync(dot_out, dd, sizeof(T), cudaMemcpyDeviceToHost, run)) != cudaSuccess) return cuda_fail(e);
    for (cudaStream_t st : d->chain_streams)
        if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(e);
    return STREAMOPS_OK;
}

}  // namespace

namespace streamops {
int note_cuda_error(cudaError_t e) { return cuda_fail(e); }
void note_launches(int n) { g_launches.fetch_add((unsigned long long)n); }
}  // namespace streamops

extern "C" {

#define STREAMOPS_UNARY(NAME, OP, T, DT)                                                             \
    int NAME(const T *x, T *out, double scalar, size_t n, streamops_stream_t stream) {               \
        return run_op(OP, DT, x, nullptr, out, scalar, n, stream);                                   \
    }
#define STREAMOPS_BINARY(NAME, OP, T, DT)                                                            \
    int NAME(const T *x, const T *y, T *out, double scalar, size_t n, streamops_stream_t stream) {   \
        return run_op(OP, DT, x, y, out, scalar, n, stream);                                         \
    }
STREAMOPS_UNARY(stream_copy_f64, OP_COPY, double, DT_F64)
STREAMOPS_UNARY(stream_copy_f32, OP_COPY, float, DT_F32)
STREAMOPS_UNARY(stream_scale_f64, OP_SCALE, double, DT_F64)
STREAMOPS_UNARY(stream_scale_f32, OP_SCALE, float, DT_F32)
STREAMOPS_BINARY(stream_add_f64, OP_ADD, double, DT_F64)
STREAMOPS_BINARY(stream_add_f32, OP_ADD, float, DT_F32)
STREAMOPS_BINARY(stream_triad_f64, OP_TRIAD, double, DT_F64)
STREAMOPS_BINARY(stream_triad_f32, OP_TRIAD, float, DT_F32)
STREAMOPS_BINARY(stream_dot_f64, OP_DOT, double, DT_F64)
STREAMOPS_BINARY(stream_dot_f32, OP_DOT, float, DT_F32)

int stream_dot_wide_f32(const float *x, const float *y, double *out, double scalar, size_t n, streamops_stream_t stream) {
    return run_op(OP_DOT, DT_F32, x, y, out, scalar, n, stream, true);
}

static int fold(int dtype, const double *partials, void *out, size_t count, streamops_stream_t stream) {
    if (!out || (count > 0 && !partials)) return STREAMOPS_ERR_NULL;
    if (((uintptr_t)partials % 8) || ((uintptr_t)out % (dtype == DT_F64 ? 8 : 4))) return STREAMOPS_ERR_ALIGN;
    if (count > ((size_t)1 << 24)) return STREAMOPS_ERR_ARG;
    if (count > 0 && ranges_overlap(partials, count * 8, out, dtype == DT_F64 ? 8 : 4)) return STREAMOPS_ERR_OVERLAP;
    cudaError_t e = launch_fold(dtype, partials, count, out, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    g_launches.fetch_add(1);
    return STREAMOPS_OK;
}
int stream_fold_f64(const double *partials, double *out, double scalar, size_t count, streamops_stream_t stream) {
    (void)scalar;
    return fold(DT_F64, partials, out, count, stream);
}
int stream_fold_f32(const double *partials, float *out, double scalar, size_t count, streamops_stream_t stream) {
    (void)scalar;
    return fold(DT_F32, partials, out, count, stream);
}

// Device-pointer chain: five asynchronous launches from one call.
static int chain_device(int dtype, void *a, void *b, void *c, void *dot_out, double scalar, size_t n,
                        streamops_stream_t stream) {
    int status;
    if ((status = run_op(OP_COPY, dtype, a, nullptr, c, scalar, n, stream)) != STREAMOPS_OK) return status;
    if ((status = run_op(OP_SCALE, dtype, c, nullptr, b, scalar, n, stream)) != STREAMOPS_OK) return status;
    if ((status = run_op(OP_ADD, dtype, a, b, c, scalar, n, stream)) != STREAMOPS_OK) return status;
    if ((status = run_op(OP_TRIAD, dtype, b, c, a, scalar, n, stream)) != STREAMOPS_OK) return status;
    return run_op(OP_DOT, dtype, a, b, dot_out, scalar, n, stream);
}
int streamops_chain_f64(double *a, double *b, double *c, double *dot_out, double scalar, size_t n,
                        streamops_stream_t stream) {
    return chain_device(DT_F64, a, b, c, dot_out, scalar, n, stream);
}
int streamops_chain_f32(float *a, float *b, float *c, float *dot_out, double scalar, size_t n,
                        streamops_stream_t stream) {
    return chain_device(DT_F32, a, b, c, dot_out, scalar, n, stream);
}

int streamops_chain_host_f64(double *a, double *b, double *c, double scalar, size_t n, double *dot_out) {
    return chain_host<double>(a, b, c, scalar, n, dot_out);
}
int streamops_chain_host_f32(float *a, float *b, float *c, double scalar, size_t n, float *dot_out) {
    return chain_host<float>(a, b, c, scalar, n, dot_out);
}

int streamops_set_host_piece_mib(int mib) {
    if (mib < 1 || mib > 4096) return STREAMOPS_ERR_ARG;
    g_chain_piece_bytes.store((size_t)mib << 20);
    return STREAMOPS_OK;
}

int streamops_init(int device) {
    DeviceState *d = nullptr;
    return init_device(device, &d);
}

int streamops_shutdown(void) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) { (void)cudaGetLastError(); return STREAMOPS_OK; }
    for (int i = 0; i < kMaxDevices; ++i) {
        DeviceState &d = g_dev[i];
        if (!d.ready) continue;
        cudaSetDevice(i);
        cudaDeviceSynchronize();
        cudaFree(d.partials); cudaFree(d.tickets); cudaFree(d.error_flag); cudaFree(d.chain_dot);
        for (void *&p : d.chain_buf) { cudaFree(p); p = nullptr; }
        cudaFree(d.chain_partials); d.chain_partials = nullptr;
        for (cudaStream_t &st : d.chain_streams) { if (st) cudaStreamDestroy(st); st = nullptr; }
        for (cudaEvent_t ev : d.chain_events) cudaEventDestroy(ev);
        d.chain_events.clear();
        d.partials = nullptr; d.tickets = nullptr; d.error_flag = nullptr; d.chain_dot = nullptr;
        d.chain_bytes = 0; d.ready = false;
    }
    cudaSetDevice(prev);
    return STREAMOPS_OK;
}

int streamops_set_tuning(int op, int dtype, const streamops_tuning_t *t) {
    if (!t) return STREAMOPS_ERR_NULL;
    if (op < 0 || op >= OP_COUNT || dtype < 0 || dtype > 1 || !valid_tuning(*t)) return STREAMOPS_ERR_ARG;
    (void)tuning(op, dtype);
    g_tuning[op][dtype] = *t;
    return STREAMOPS_OK;
}

int streamops_get_tuning(int op, int dtype, streamops_tuning_t *t) {
    if (!t) return STREAMOPS_ERR_NULL;
    if (op < 0 || op >= OP_COUNT || dtype < 0 || dtype > 1) return STREAMOPS_ERR_ARG;
    *t = tuning(op, dtype);
    return STREAMOPS_OK;
}

int streamops_reset_tuning(void) {
    (void)tuning(0, 0);
    init_tuning();
    return STREAMOPS_OK;
}

const char *streamops_policy_name(int policy) {
    switch (policy) {
        case 0: return "ld.global / st.global";
        case 1: return "ld.global.nc / st.global";
        case 2: return "ld.global.cs / st.global.cs";
        case 3: return "ld.global.L1::no_allocate / st.global.cs";
        case 4: return "ld.global.L1::no_allocate + L2 evict_first / st.global + L2 evict_first";
        case 5: return "ld.global.L1::no_allocate + L2 evict_first / st.global";
        case 6: return "ld.global.L1::no_allocate + L2 evict_first / st.global + L2 evict_last";
        case 7: return "ld.global.L1::no_allocate + L2 evict_first / st.global + L2 evict_first, plain st.global for the last keep_mib MiB";
        case 8: return "ld.global.L1::no_allocate + L2 evict_first / st.global + L2 evict_first, evict_last for the last keep_mib MiB";
        default: return "unknown";
    }
}

int streamops_check(streamops_stream_t stream) {
    DeviceState *d = nullptr;
    int status = current_device_state(&d);
    if (status != STREAMOPS_OK) return status;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    int flag = 0;
    if ((e = cudaMemcpy(&flag, d->error_flag, sizeof(int), cudaMemcpyDeviceToHost)) != cudaSuccess) return cuda_fail(e);
    if (flag == 0) return STREAMOPS_OK;
    if ((e = cudaMemset(d->error_flag, 0, sizeof(int))) != cudaSuccess) return cuda_fail(e);
    return STREAMOPS_ERR_TIMEOUT;
}

const char *streamops_status_string(int status) {
    switch (status) {
        case STREAMOPS_OK: return "ok";
        case STREAMOPS_ERR_NULL: return "null pointer";
        case STREAMOPS_ERR_ALIGN: return "pointer not aligned to the element size";
        case STREAMOPS_ERR_OVERLAP: return "output partially overlaps an input";
        case STREAMOPS_ERR_CUDA: return "CUDA error (see streamops_last_cuda_error)";
        case STREAMOPS_ERR_WORKSPACE: return "workspace allocation failed";
        case STREAMOPS_ERR_TIMEOUT: return "a bounded wait inside a kernel gave up";
        case STREAMOPS_ERR_ARG: return "argument out of range";
        case STREAMOPS_ERR_TOO_LARGE: return "n exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

int streamops_last_cuda_error(void) { return g_last_cuda_error.load(); }

unsigned long long streamops_launch_count(void) { return g_launches.load(); }

}  // extern "C"
