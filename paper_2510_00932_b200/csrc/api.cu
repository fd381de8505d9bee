// The C ABI of libstreamops: argument checks, per-device state, tuning table, dispatch.
// Declarations and the contract of every entry point are in include/streamops.h.
#include <atomic>
#include <cstring>
#include <initializer_list>
#include <mutex>

#include "../../include/streamops.h"
#include "indexcheck.cuh"
#include "internal.cuh"

using namespace streamops;

namespace {

constexpr int kMaxDevices = 64;
constexpr int kChainRing = 4;           // stages of the host-buffer pipeline: pieces in flight

// One Dot workspace slot of a device. A slot belongs to the stream that used it last: that stream
// may use it again at once (its Dots run in stream order); another stream may take it over only
// when the slot's last Dot has finished. Every Dot gets the next sequence number of its slot
// (`issued`), and the block that finishes it writes that number into the high half of the slot's
// ticket word as its last act: the slot is idle when the two agree. Nothing is added to the stream
// between kernels (an event record there would end the overlap of dependent launches).
struct DotSlot {
    cudaStream_t owner = nullptr;
    unsigned issued = 0;
    bool used = false;
};

struct DeviceState {
    std::atomic<bool> ready{false};
    int sm_count = 0;
    double *partials = nullptr;        // kDotSlots * kMaxDotBlocks doubles
    unsigned long long *tickets = nullptr;   // kDotSlots ticket words (see DotScratch), low halves zero between calls
    int *error_flag = nullptr;         // set by a bounded wait that gave up
    unsigned long long *done_host = nullptr;   // pinned host copy of the ticket words, refreshed only when a slot has to change hands
    cudaStream_t probe_stream = nullptr;   // carries that refresh, so that no caller's stream is touched
    std::mutex slot_mutex;
    DotSlot slots[kDotLiveSlots];      // slots of ordinary calls; the rest serve stream capture
    unsigned steal_cursor = 0;
    std::atomic<unsigned> next_capture_slot{0};
    // the array most recently written by an elementwise kernel on this device and the end of it that
    // was written last (1 = high addresses): where its still-cached lines are. Packed into atomics;
    // a stale or torn reading only costs bandwidth.
    std::atomic<uintptr_t> last_written{0};
    std::atomic<size_t> last_written_bytes{0};
    std::atomic<int> last_written_end_high{0};
    // host-path ring (streamops_chain_host_*)
    std::mutex chain_mutex;                            // one host-buffer pass per device at a time
    void *chain_ring = nullptr;                        // kChainRing stages of three piece buffers each
    size_t chain_piece_bytes = 0;                      // bytes of one piece buffer in the ring
    void *chain_dot = nullptr;
    double *chain_partials = nullptr;                  // one double per piece
    cudaStream_t chain_streams[3] = {nullptr, nullptr, nullptr};   // upload, kernels, download
    cudaEvent_t chain_uploaded[kChainRing] = {}, chain_computed[kChainRing] = {}, chain_downloaded[kChainRing] = {};
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
    t.policy = 7; t.contiguous = 0; t.chunk_bytes = 16384; t.stages = 4; t.two_pass = 0; t.reverse = 0; t.pdl = 1; t.keep_mib = 112; t.compensated = 0; t.pipeline = 0;
    const bool f64 = dtype == DT_F64;
    switch (op) {
        case OP_COPY:  t.reverse = 2; break;
        case OP_SCALE: t.reverse = 2; break;
        case OP_ADD:   t.threads = 128; t.reverse = 2; break;
        case OP_TRIAD: t.threads = 128; t.reverse = 2; break;
        // Dot, double: the rolling-slot kernel with two slots per thread on two blocks per SM (measured
        // against the tile-at-a-time kernel: 77.4 vs 78.4 us at n = 2^25, equal at 2^28, 9.7 vs 12.4 us at
        // 2^22); float: tiles of two vectors on two blocks per SM measured best from 16 MiB to 2 GiB
        case OP_DOT:
            t.threads = 512; t.policy = 4; t.unroll = 2;
            t.pipeline = f64 ? 1 : 0; t.blocks_per_sm = f64 ? 0 : 2;
            break;
    }
    return t;
}

// The tuning table. Readers take a copy under the mutex, so a call that runs while another thread
// changes the table sees either the old or the new entry, never a mixture.
streamops_tuning_t g_tuning[OP_COUNT][2];
bool g_tuning_ready = false;
std::mutex g_tuning_mutex;
void init_tuning_locked() {
    for (int op = 0; op < OP_COUNT; ++op)
        for (int dt = 0; dt < 2; ++dt) g_tuning[op][dt] = default_tuning(op, dt);
    g_tuning_ready = true;
}
streamops_tuning_t tuning(int op, int dtype) {
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    if (!g_tuning_ready) init_tuning_locked();
    return g_tuning[op][dtype];
}
std::atomic<unsigned> g_wait_limit{1u << 22};   // mbarrier.try_wait attempts of the bulk pipelines

int cuda_fail(cudaError_t e) {
    g_last_cuda_error.store((int)e);
    return STREAMOPS_ERR_CUDA;
}

void free_workspace(DeviceState &d) {
    cudaFree(d.partials); cudaFree(d.tickets); cudaFree(d.error_flag);
    if (d.done_host) cudaFreeHost(d.done_host);
    if (d.probe_stream) cudaStreamDestroy(d.probe_stream);
    d.partials = nullptr; d.tickets = nullptr; d.error_flag = nullptr;
    d.done_host = nullptr; d.probe_stream = nullptr;
    for (DotSlot &s : d.slots) s = DotSlot{};
}

int init_device(int device, DeviceState **out) {
    if (device < 0 || device >= kMaxDevices) return STREAMOPS_ERR_ARG;
    DeviceState &d = g_dev[device];
    if (!d.ready.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!d.ready.load(std::memory_order_relaxed)) {
            int prev = 0;
            cudaError_t e = cudaGetDevice(&prev);
            if (e != cudaSuccess) return cuda_fail(e);
            if ((e = cudaSetDevice(device)) != cudaSuccess) return cuda_fail(e);
            int status = STREAMOPS_OK;
            do {
                if ((e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess) { status = cuda_fail(e); break; }
                const size_t pbytes = sizeof(double) * kDotSlots * kMaxDotBlocks;
                if (cudaMalloc(&d.partials, pbytes) != cudaSuccess ||
                    cudaMalloc(&d.tickets, sizeof(unsigned long long) * kDotSlots) != cudaSuccess ||
                    cudaMalloc(&d.error_flag, sizeof(int)) != cudaSuccess ||
                    cudaMallocHost(&d.done_host, sizeof(unsigned long long) * kDotLiveSlots) != cudaSuccess) {
                    (void)cudaGetLastError();
                    status = STREAMOPS_ERR_WORKSPACE; break;
                }
                if ((e = cudaMemset(d.tickets, 0, sizeof(unsigned long long) * kDotSlots)) != cudaSuccess) { status = cuda_fail(e); break; }
                if ((e = cudaMemset(d.error_flag, 0, sizeof(int))) != cudaSuccess) { status = cuda_fail(e); break; }
                if ((e = cudaStreamCreateWithFlags(&d.probe_stream, cudaStreamNonBlocking)) != cudaSuccess) { status = cuda_fail(e); break; }
                for (DotSlot &s : d.slots) s = DotSlot{};
            } while (false);
            if (status != STREAMOPS_OK) {
                free_workspace(d);
                cudaSetDevice(prev);
                return status;
            }
            cudaSetDevice(prev);
            d.ready.store(true, std::memory_order_release);
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
    c.pipeline = (op == OP_DOT && t.pipeline && c.vec_bytes == 32 && c.unroll >= 2) ? 1 : 0;
    c.policy = t.policy;
    // the read-only data path must not be used on an array the kernel also writes
    if (c.policy == 1 && (out == x || out == y)) c.policy = 0;
    if (op == OP_DOT && c.policy > 6) c.policy = 4;           // Dot stores nothing: the two-phase sets reduce to 4
    const size_t per_tile = (size_t)c.threads * (c.vec_bytes ? (size_t)(c.pipeline ? 1 : c.unroll) * c.vec_bytes / esize : 1);
    const size_t tiles = (n + per_tile - 1) / per_tile;
    size_t grid = t.blocks_per_sm > 0 ? (size_t)t.blocks_per_sm * d.sm_count : tiles;
    if (op == OP_DOT && t.blocks_per_sm == 0 && c.pipeline) {
        grid = (size_t)2 * d.sm_count;                           // the rolling-slot kernel keeps two blocks per SM busy
    } else if (op == OP_DOT && t.blocks_per_sm == 0) {
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
    if (t.pipeline != 0 && t.pipeline != 1) return false;
    if (t.chunk_bytes < 1024 || t.chunk_bytes > 65536 || (t.chunk_bytes & 15)) return false;
    if (t.stages < 2 || t.stages > 8) return false;
    if (t.reverse < 0 || t.reverse > 2) return false;
    return true;
}

// Picks the workspace slot of one Dot call on `stream` and fills in its scratch pointers.
// Ordinary calls: the slot this stream used last (stream order makes reuse safe), else a slot never
// used, else a slot whose last Dot has finished (the ticket words are copied to the host on a stream
// of the library's own: this is the only path that waits for anything, and only for that copy); if
// all kDotLiveSlots slots are still in flight on other streams, STREAMOPS_ERR_WORKSPACE.
// Calls made while `stream` is being captured: one of the kDotCaptureSlots slots set aside for graphs,
// handed out in turn and never shared with ordinary calls; the slot is baked into the graph.
int acquire_dot_slot(DeviceState *d, cudaStream_t stream, DotScratch *scratch, DotSlot **live) {
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    cudaError_t e = cudaStreamIsCapturing(stream, &capturing);
    if (e != cudaSuccess) return cuda_fail(e);
    *live = nullptr;
    int found = -1;
    if (capturing != cudaStreamCaptureStatusNone) {
        found = kDotLiveSlots + (int)(d->next_capture_slot.fetch_add(1) % (unsigned)kDotCaptureSlots);
        scratch->seq = 0;
    } else {
        std::lock_guard<std::mutex> lock(d->slot_mutex);
        for (int i = 0; i < kDotLiveSlots && found < 0; ++i)
            if (d->slots[i].used && d->slots[i].owner == stream) found = i;
        for (int i = 0; i < kDotLiveSlots && found < 0; ++i)
            if (!d->slots[i].used) found = i;
        if (found < 0) {
            if ((e = cudaMemcpyAsync(d->done_host, d->tickets, sizeof(unsigned long long) * kDotLiveSlots, cudaMemcpyDeviceToHost,
                                     d->probe_stream)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaStreamSynchronize(d->probe_stream)) != cudaSuccess) return cuda_fail(e);
            for (int k = 0; k < kDotLiveSlots && found < 0; ++k) {
                const int i = (int)((d->steal_cursor + (unsigned)k) % (unsigned)kDotLiveSlots);
                // finished: the high half carries the last issued number (and the ticket is back at zero)
                if (d->done_host[i] == ((unsigned long long)d->slots[i].issued << 32)) { found = i; d->steal_cursor = (unsigned)i + 1; }
            }
        }
        if (found < 0) return STREAMOPS_ERR_WORKSPACE;
        DotSlot &s = d->slots[found];
        s.used = true;
        s.owner = stream;
        scratch->seq = ++s.issued;
        *live = &s;
    }
    scratch->partials = d->partials + (size_t)found * kMaxDotBlocks;
    scratch->ticket = d->tickets + found;
    return STREAMOPS_OK;
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
    const streamops_tuning_t t = tuning(op, dtype);

    DotScratch scratch{nullptr, nullptr, 0};
    DotSlot *live_slot = nullptr;
    if (op == OP_DOT && (status = acquire_dot_slot(d, stream, &scratch, &live_slot)) != STREAMOPS_OK) return status;

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
        b.wait_limit = g_wait_limit.load();
        const size_t nchunks = (n * esize + b.chunk_bytes - 1) / b.chunk_bytes;
        size_t grid = (size_t)(t.blocks_per_sm > 0 ? t.blocks_per_sm : 1) * d->sm_count;
        if (grid > nchunks) grid = nchunks;
        if (op == OP_DOT && grid > (size_t)kMaxDotBlocks) grid = kMaxDotBlocks;
        b.grid = clamp_grid(grid);
        e = launch_bulk(op, dtype, b, x, y, out, scalar, n, scratch, d->error_flag, stream, &launches);
    } else {
        VecLaunch c = resolve_vec(t, *d, op, esize, x, y, out, n);
        if (op != OP_DOT) {
            // is an input of this call the array the previous elementwise kernel on the device wrote?
            const uintptr_t w = d->last_written.load();
            const bool consumer = w != 0 && d->last_written_bytes.load() == n * esize &&
                                  (w == (uintptr_t)x || (uses_y && w == (uintptr_t)y));
            // automatic direction: a consumer starts at the end its producer wrote last (those lines are
            // the ones still in L2)
            if (t.reverse == 2) c.reverse = consumer && d->last_written_end_high.load() != 0;
            // two-phase stores keep the end of the output in L2 for a consumer. A call that is itself a
            // consumer is a link of a dataflow chain, so its output is likely to be read next; a call
            // that is not gets streaming (evict-first) stores throughout, which is the faster choice
            // when nobody comes for the output
            if ((c.policy == 7 || c.policy == 8) && !consumer) c.policy = 4;
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
    if (e != cudaSuccess) {
        if (live_slot) {                                  // nothing was launched: the slot's count goes back
            std::lock_guard<std::mutex> lock(d->slot_mutex);
            --live_slot->issued;
        }
        return cuda_fail(e);
    }
    g_launches.fetch_add((unsigned long long)launches);
    return STREAMOPS_OK;
}

// Host-buffer pass, pipelined through a small ring of device buffers: the arrays are cut into pieces
// of g_chain_piece_bytes per array; piece k of a (the pass's only input: b and c are overwritten before
// they are read) is uploaded into ring stage k mod kChainRing on one
// stream, run through the five kernels on a second (Dot as a double partial sum per piece), and
// downloaded on a third, so that uploads, kernels and downloads of different pieces overlap and the
// two directions of the host link are busy at the same time. A stage is refilled only after the
// download of the piece that used it before has finished (an event per stage). Device memory
// needed: kChainRing x 3 piece buffers, whatever n is. The dot product is the left-to-right fold of
// the per-piece partial sums: fixed by n and the piece size alone, so repeatable bit for bit.
std::atomic<size_t> g_chain_piece_bytes{(size_t)16 << 20};
constexpr size_t kChainMaxPieces = 4096;

template <typename T>
int chain_host(T *a, T *b, T *c, double scalar, size_t n, T *dot_out) {
    constexpr int dtype = sizeof(T) == 8 ? DT_F64 : DT_F32;
    if (!dot_out || (n > 0 && (!a || !b || !c))) return STREAMOPS_ERR_NULL;
    DeviceState *d = nullptr;
    int status = current_device_state(&d);
    if (status != STREAMOPS_OK) return status;
    cudaError_t e;
    cudaEvent_t end_run = nullptr, end_down = nullptr;
    {
        // issuing is serialised per device; the lock is released before the host waits, and a second
        // caller's work simply queues behind this one's on the same three streams
        std::lock_guard<std::mutex> lock(d->chain_mutex);
        for (cudaStream_t &st : d->chain_streams)
            if (!st && (e = cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
        for (int s = 0; s < kChainRing; ++s)
            for (cudaEvent_t *ev : {&d->chain_uploaded[s], &d->chain_computed[s], &d->chain_downloaded[s]})
                if (!*ev && (e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        if (!d->chain_dot && (cudaMalloc(&d->chain_dot, 8) != cudaSuccess ||
                              cudaMalloc(&d->chain_partials, sizeof(double) * kChainMaxPieces) != cudaSuccess)) {
            (void)cudaGetLastError();
            return STREAMOPS_ERR_WORKSPACE;
        }
        // pieces of equal length (the last one shorter), at most kChainMaxPieces of them. (Shorter first
        // and last pieces were measured and change nothing: filling and draining the pipeline is not where
        // the time against the link's own rate goes.)
        size_t piece = g_chain_piece_bytes.load() / sizeof(T);
        while ((n + piece - 1) / piece > kChainMaxPieces) piece *= 2;
        const size_t pieces = n ? (n + piece - 1) / piece : 0;
        const size_t piece_bytes = piece * sizeof(T);
        cudaStream_t up = d->chain_streams[0], run = d->chain_streams[1], down = d->chain_streams[2];
        if (piece_bytes != d->chain_piece_bytes) {
            // a ring of another piece size: wait for whatever still uses the old one, then replace it
            for (cudaStream_t st : d->chain_streams)
                if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(e);
            cudaFree(d->chain_ring); d->chain_ring = nullptr; d->chain_piece_bytes = 0;
            if (cudaMalloc(&d->chain_ring, piece_bytes * 3 * kChainRing) != cudaSuccess) {
                (void)cudaGetLastError();
                return STREAMOPS_ERR_WORKSPACE;
            }
            d->chain_piece_bytes = piece_bytes;
        }
        T *host[3] = {a, b, c};
        T *dd = (T *)d->chain_dot;
        for (size_t k = 0; k < pieces; ++k) {
            const size_t lo = k * piece, len = n - lo < piece ? n - lo : piece;
            const int s = (int)(k % kChainRing);
            T *dev[3];
            for (int i = 0; i < 3; ++i) dev[i] = (T *)((char *)d->chain_ring + ((size_t)s * 3 + i) * piece_bytes);
            // the stage is free once the download of its previous piece (this call's or an earlier
            // call's) has finished; an event that was never recorded counts as complete
            if ((e = cudaStreamWaitEvent(up, d->chain_downloaded[s], 0)) != cudaSuccess) return cuda_fail(e);
            // only a travels to the device: the pass overwrites c (c <- a) and b (b <- s*c) before it reads
            // them, so their contents on entry are no inputs of the computation
            if ((e = cudaMemcpyAsync(dev[0], host[0] + lo, len * sizeof(T), cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventRecord(d->chain_uploaded[s], up)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaStreamWaitEvent(run, d->chain_uploaded[s], 0)) != cudaSuccess) return cuda_fail(e);
            T *pa = dev[0], *pb = dev[1], *pc = dev[2];
            // c <- a; b <- s*c; c <- a+b; a <- b+s*c; partial dot(a, b)
            if ((status = run_op(OP_COPY, dtype, pa, nullptr, pc, scalar, len, run)) != STREAMOPS_OK) return status;
            if ((status = run_op(OP_SCALE, dtype, pc, nullptr, pb, scalar, len, run)) != STREAMOPS_OK) return status;
            if ((status = run_op(OP_ADD, dtype, pa, pb, pc, scalar, len, run)) != STREAMOPS_OK) return status;
            if ((status = run_op(OP_TRIAD, dtype, pb, pc, pa, scalar, len, run)) != STREAMOPS_OK) return status;
            if ((status = run_op(OP_DOT, dtype, pa, pb, d->chain_partials + k, scalar, len, run, dtype == DT_F32)) != STREAMOPS_OK) return status;
            if ((e = cudaEventRecord(d->chain_computed[s], run)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaStreamWaitEvent(down, d->chain_computed[s], 0)) != cudaSuccess) return cuda_fail(e);
            for (int i = 0; i < 3; ++i)
                if ((e = cudaMemcpyAsync(host[i] + lo, dev[i], len * sizeof(T), cudaMemcpyDeviceToHost, down)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventRecord(d->chain_downloaded[s], down)) != cudaSuccess) return cuda_fail(e);
        }
        if ((e = launch_fold(dtype, d->chain_partials, pieces, dd, run)) != cudaSuccess) return cuda_fail(e);
        g_launches.fetch_add(1);
        if ((e = cudaMemcpyAsync(dot_out, dd, sizeof(T), cudaMemcpyDeviceToHost, run)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&end_run, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&end_down, cudaEventDisableTiming)) != cudaSuccess) { cudaEventDestroy(end_run); return cuda_fail(e); }
        e = cudaEventRecord(end_run, run);
        if (e == cudaSuccess) e = cudaEventRecord(end_down, down);
        if (e != cudaSuccess) { cudaEventDestroy(end_run); cudaEventDestroy(end_down); return cuda_fail(e); }
    }
    // this call's own work only: the kernels and the dot product, then the last download
    e = cudaEventSynchronize(end_run);
    const cudaError_t e2 = cudaEventSynchronize(end_down);
    cudaEventDestroy(end_run);
    cudaEventDestroy(end_down);
    if (e != cudaSuccess) return cuda_fail(e);
    if (e2 != cudaSuccess) return cuda_fail(e2);
    return STREAMOPS_OK;
}

}  // namespace

namespace streamops {
// Readers of the per-translation-unit index-violation records (checking builds register one per
// kernel file during static initialisation; an ordinary build registers none).
namespace {
constexpr int kMaxViolationReaders = 16;
violation_reader_t g_violation_readers[kMaxViolationReaders];
int g_violation_reader_count = 0;
}  // namespace
void register_violation_reader(violation_reader_t reader) {
    if (g_violation_reader_count < kMaxViolationReaders) g_violation_readers[g_violation_reader_count++] = reader;
}
int note_cuda_error(cudaError_t e) { return cuda_fail(e); }
void note_launches(int n) { g_launches.fetch_add((unsigned long long)n); }
}  // namespace streamops

#ifdef STREAMOPS_CHECK_INDICES
// Asks index_ok about an access that does not fit, without making any access: exercises the record.
__global__ void index_selftest_kernel(unsigned long long offset, unsigned long long width, unsigned long long limit, int *verdicts) {
    verdicts[0] = index_ok((size_t)offset, (size_t)width, (size_t)limit, W_SELFTEST) ? 1 : 0;
    verdicts[1] = index_ok((size_t)(limit - width), (size_t)width, (size_t)limit, W_SELFTEST) ? 1 : 0;
}
#endif

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

int stream_dot_timeline_f64(const double *x, const double *y, double *out, size_t n, streamops_stream_t stream_,
                            unsigned long long *stamps, unsigned *blocks) {
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!stamps || !blocks) return STREAMOPS_ERR_NULL;
    int status = check_args(OP_DOT, 8, x, y, out, n, 8);
    if (status != STREAMOPS_OK) return status;
    if (n == 0 || (((uintptr_t)x | (uintptr_t)y) & 31)) return STREAMOPS_ERR_ARG;     // the 32-byte-vector kernel only
    DeviceState *d = nullptr;
    if ((status = current_device_state(&d)) != STREAMOPS_OK) return status;
    streamops_tuning_t t = default_tuning(OP_DOT, DT_F64);
    const VecLaunch c = resolve_vec(t, *d, OP_DOT, 8, x, y, out, n);
    if (c.grid > (unsigned)STREAMOPS_TIMELINE_MAX_BLOCKS) return STREAMOPS_ERR_ARG;
    DotScratch scratch{nullptr, nullptr, 0};
    DotSlot *live_slot = nullptr;
    if ((status = acquire_dot_slot(d, stream, &scratch, &live_slot)) != STREAMOPS_OK) return status;
    const cudaError_t e = launch_dot_timeline(c, x, y, out, n, scratch, stamps, stream);
    if (e != cudaSuccess) {
        if (live_slot) {
            std::lock_guard<std::mutex> lock(d->slot_mutex);
            --live_slot->issued;
        }
        return cuda_fail(e);
    }
    *blocks = c.grid;
    g_launches.fetch_add(1);
    return STREAMOPS_OK;
}

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
        if (!d.ready.load(std::memory_order_acquire)) continue;
        cudaSetDevice(i);
        cudaDeviceSynchronize();
        free_workspace(d);
        cudaFree(d.chain_dot);
        cudaFree(d.chain_ring); d.chain_ring = nullptr; d.chain_piece_bytes = 0;
        cudaFree(d.chain_partials); d.chain_partials = nullptr;
        for (cudaStream_t &st : d.chain_streams) { if (st) cudaStreamDestroy(st); st = nullptr; }
        for (int s = 0; s < kChainRing; ++s)
            for (cudaEvent_t *ev : {&d.chain_uploaded[s], &d.chain_computed[s], &d.chain_downloaded[s]}) {
                if (*ev) cudaEventDestroy(*ev);
                *ev = nullptr;
            }
        d.chain_dot = nullptr;
        d.last_written.store(0);
        d.ready.store(false, std::memory_order_release);
    }
    cudaSetDevice(prev);
    return STREAMOPS_OK;
}

int streamops_set_tuning(int op, int dtype, const streamops_tuning_t *t) {
    if (!t) return STREAMOPS_ERR_NULL;
    if (op < 0 || op >= OP_COUNT || dtype < 0 || dtype > 1 || !valid_tuning(*t)) return STREAMOPS_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    if (!g_tuning_ready) init_tuning_locked();
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
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    init_tuning_locked();
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
        case 7: return "ld.global.L1::no_allocate + L2 evict_first / st.global + L2 evict_first, plain st.global for the last keep_mib MiB when the call consumes the previous call's output";
        case 8: return "ld.global.L1::no_allocate + L2 evict_first / st.global + L2 evict_first, evict_last for the last keep_mib MiB when the call consumes the previous call's output";
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
        case STREAMOPS_ERR_WORKSPACE: return "workspace unavailable (allocation failed, or every Dot slot is in flight)";
        case STREAMOPS_ERR_TIMEOUT: return "a bounded wait inside a kernel gave up";
        case STREAMOPS_ERR_ARG: return "argument out of range";
        case STREAMOPS_ERR_TOO_LARGE: return "n exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

int streamops_set_wait_limit(unsigned tries) {
    g_wait_limit.store(tries == 0 ? (1u << 22) : tries);
    return STREAMOPS_OK;
}

int streamops_index_violation(int *where, unsigned long long *offset, unsigned long long *limit) {
#ifdef STREAMOPS_CHECK_INDICES
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return -cuda_fail(e);
    for (int i = 0; i < g_violation_reader_count; ++i) {
        IndexViolation v{0, 0, 0, 0};
        if ((e = g_violation_readers[i](&v, true)) != cudaSuccess) return -cuda_fail(e);
        if (v.flag) {
            if (where) *where = v.where;
            if (offset) *offset = v.offset;
            if (limit) *limit = v.limit;
            return 1;
        }
    }
    return 0;
#else
    (void)where; (void)offset; (void)limit;
    return -STREAMOPS_ERR_ARG;            // not a checking build
#endif
}

int streamops_index_selftest(unsigned long long offset, unsigned long long width, unsigned long long limit) {
#ifdef STREAMOPS_CHECK_INDICES
    if (width == 0 || width > limit) return -STREAMOPS_ERR_ARG;
    int *verdicts = nullptr;
    if (cudaMalloc(&verdicts, 2 * sizeof(int)) != cudaSuccess) { (void)cudaGetLastError(); return -STREAMOPS_ERR_WORKSPACE; }
    index_selftest_kernel<<<1, 1>>>(offset, width, limit, verdicts);
    int host[2] = {-1, -1};
    cudaError_t e = cudaMemcpy(host, verdicts, sizeof host, cudaMemcpyDeviceToHost);
    cudaFree(verdicts);
    if (e != cudaSuccess) return -cuda_fail(e);
    return host[0] | (host[1] << 1);       // bit 0: the probed access was accepted; bit 1: the last fitting access was
#else
    (void)offset; (void)width; (void)limit;
    return -STREAMOPS_ERR_ARG;
#endif
}

int streamops_last_cuda_error(void) { return g_last_cuda_error.load(); }

unsigned long long streamops_launch_count(void) { return g_launches.load(); }

}  // extern "C"
