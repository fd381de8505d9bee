/*
 * libstreamops -- the memory-bound streaming kernels Copy, Mul (scale), Add, Triad and Dot for
 * NVIDIA B200 (sm_100a), behind a plain C ABI.
 *
 * The kernels are the five STREAM-style vector operations the paper evaluates (Table 1:
 * "Copy", "Mul", "Add", "Triad", "Dot"; Section 5.2). The paper names them without printing a
 * formula; each entry point below states the textbook definition it implements.
 *
 * Conventions for every stream_* entry point
 *   - x, y, out are DEVICE pointers on the current device to dense, contiguous 1-D arrays of n
 *     elements (out of Dot: one element). The caller owns them; the library never frees,
 *     reallocates or keeps them.
 *   - The call is asynchronous on `stream` (a cudaStream_t passed as a pointer; NULL is the
 *     default stream). No call synchronises the host, copies to the host, or allocates, except
 *     the one-time per-device workspace described under streamops_init.
 *   - `scalar` is rounded once, to nearest-even, to the element type before use. Copy, Add and
 *     Dot ignore it (one uniform signature).
 *   - Arithmetic is IEEE-754 round-to-nearest-even in the element type, subnormals honoured,
 *     one rounding per operation: Triad is a rounded multiply followed by a rounded add, never
 *     a fused multiply-add. The four elementwise kernels therefore have exactly one correct
 *     bit pattern per element (NaN payloads aside; Copy preserves every bit pattern).
 *   - Pointers must be aligned to the element size; 16- or 32-byte alignment selects the
 *     vector kernels, anything else runs the scalar kernel with identical results.
 *   - out may be exactly x or exactly y (in place). Any other overlap of out with an input is
 *     rejected with STREAMOPS_ERR_OVERLAP.
 *   - n == 0 is valid and touches no element (Dot writes +0).
 *   - Return value: a STREAMOPS_* status. Nothing throws, aborts or prints.
 */
#ifndef STREAMOPS_H
#define STREAMOPS_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void *streamops_stream_t; /* a cudaStream_t */

enum streamops_status {
    STREAMOPS_OK = 0,
    STREAMOPS_ERR_NULL = 1,      /* a null pointer with n > 0 */
    STREAMOPS_ERR_ALIGN = 2,     /* a pointer not aligned to the element size */
    STREAMOPS_ERR_OVERLAP = 3,   /* out partially overlaps an input */
    STREAMOPS_ERR_CUDA = 4,      /* a CUDA call failed; see streamops_last_cuda_error */
    STREAMOPS_ERR_WORKSPACE = 5, /* the per-device workspace could not be created, or every Dot slot is in flight */
    STREAMOPS_ERR_TIMEOUT = 6,   /* a bounded wait inside a bulk-copy kernel gave up */
    STREAMOPS_ERR_ARG = 7,       /* an argument outside its documented range */
    STREAMOPS_ERR_TOO_LARGE = 8  /* n exceeds what the fixed scratch of stream_dot_noalloc_f64 covers */
};

enum streamops_op { STREAMOPS_COPY = 0, STREAMOPS_SCALE = 1, STREAMOPS_ADD = 2,
                    STREAMOPS_TRIAD = 3, STREAMOPS_DOT = 4 };
enum streamops_dtype { STREAMOPS_F32 = 0, STREAMOPS_F64 = 1 };

/* Copy (Table 1, "Copy"): out[i] = x[i] for 0 <= i < n, bit for bit (NaN payloads, signed
 * zeros and subnormals preserved). Moves 2*n*sizeof(T) bytes. */
int stream_copy_f64(const double *x, double *out, double scalar, size_t n, streamops_stream_t stream);
int stream_copy_f32(const float *x, float *out, double scalar, size_t n, streamops_stream_t stream);

/* Mul (Table 1, "Mul"; exported as "scale"): out[i] = RN(s * x[i]), s = (T)scalar.
 * Moves 2*n*sizeof(T) bytes. */
int stream_scale_f64(const double *x, double *out, double scalar, size_t n, streamops_stream_t stream);
int stream_scale_f32(const float *x, float *out, double scalar, size_t n, streamops_stream_t stream);

/* Add (Table 1, "Add"): out[i] = RN(x[i] + y[i]). Moves 3*n*sizeof(T) bytes. */
int stream_add_f64(const double *x, const double *y, double *out, double scalar, size_t n, streamops_stream_t stream);
int stream_add_f32(const float *x, const float *y, float *out, double scalar, size_t n, streamops_stream_t stream);

/* Triad (Table 1, "Triad"): out[i] = RN(x[i] + RN(s * y[i])), s = (T)scalar; two roundings.
 * Moves 3*n*sizeof(T) bytes. */
int stream_triad_f64(const double *x, const double *y, double *out, double scalar, size_t n, streamops_stream_t stream);
int stream_triad_f32(const float *x, const float *y, float *out, double scalar, size_t n, streamops_stream_t stream);

/* Dot (Table 1, "Dot"): out[0] = (T) sum_i x[i]*y[i]. out is a DEVICE pointer to one element;
 * the result stays on the device. Products and sums are carried in double for both element
 * types (a float*float product is exact in double) and rounded once to T at the end. The
 * summation order is a fixed function of n and the tuning in force -- never of block arrival
 * order or of the stream -- so repeated calls return identical bits. Accuracy: within relative
 * 1e-12 (double) / 1e-5 (float) of the exactly rounded dot product for the documented
 * workloads. Reads 2*n*sizeof(T) bytes.
 * Workspace slots. Every Dot in flight needs a slot of the per-device workspace to itself. A stream
 * keeps the slot it used last (its Dots run one after the other); a Dot on another stream takes a
 * slot that was never used or whose last Dot has finished (the finishing kernel leaves a mark in
 * device memory; when a slot has to change hands the call reads those marks with a small copy on a
 * stream of the library's own and waits for that copy only, never for a caller's stream). When all
 * STREAMOPS_DOT_SLOTS slots hold Dots still in flight on other streams the call launches nothing and
 * returns STREAMOPS_ERR_WORKSPACE: wait for one of them and call again. It never shares a slot.
 * Stream capture. A Dot issued while `stream` is being captured gets one of
 * STREAMOPS_DOT_CAPTURE_SLOTS slots set aside for graphs (handed out in turn, never used by ordinary
 * calls), and that slot is part of the captured launch: replays of one graph are safe against every
 * ordinary call; two graphs replayed at the same time are safe against each other unless more than
 * STREAMOPS_DOT_CAPTURE_SLOTS Dots have been captured in the process, after which slots repeat. A
 * captured elementwise launch likewise keeps the traversal direction chosen at capture time (see
 * `reverse` below); that affects speed only. */
int stream_dot_f64(const double *x, const double *y, double *out, double scalar, size_t n, streamops_stream_t stream);
int stream_dot_f32(const float *x, const float *y, float *out, double scalar, size_t n, streamops_stream_t stream);
#define STREAMOPS_DOT_SLOTS 24
#define STREAMOPS_DOT_CAPTURE_SLOTS 8

/* The two pieces a Dot over an array that is split across GPUs is made of (the sum is the only step
 * of the five kernels that needs an exchange: one double per GPU).
 * stream_dot_wide_f32: Dot of float arrays whose DEVICE output is the double-precision total before
 * its final rounding to float, so that per-GPU partial results lose nothing (for double arrays
 * stream_dot_f64 already is that). Always runs its second pass as a second launch.
 * stream_fold_{f64,f32}: out[0] = (T)(((p[0] + p[1]) + p[2]) + ... + p[count-1]), the doubles added
 * strictly left to right by one thread and rounded once to T: every GPU that folds the same
 * gathered partial sums in rank order gets identical bits. count <= 2^24; count == 0 writes +0. */
int stream_dot_wide_f32(const float *x, const float *y, double *out, double scalar, size_t n, streamops_stream_t stream);
int stream_fold_f64(const double *partials, double *out, double scalar, size_t count, streamops_stream_t stream);
int stream_fold_f32(const double *partials, float *out, double scalar, size_t count, streamops_stream_t stream);

/* The default double-precision Dot (same kernel, launch shape and result as stream_dot_f64 under the default
 * tuning) instrumented for profiling: thread 0 of block b stores three readings of the GPU's global
 * nanosecond timer into stamps[3 b .. 3 b + 2] -- after the wait for the previous kernel of the stream, after
 * the block's last multiply-add (all its data has arrived), and at the block's end (for the block that
 * finishes the Dot: after the final fold and the write of out[0]). stamps is a DEVICE array of at least
 * 3 * STREAMOPS_TIMELINE_MAX_BLOCKS entries; *blocks (HOST) receives the number of blocks launched. x and y
 * must be 32-byte aligned and n > 0 (STREAMOPS_ERR_ARG otherwise). `python -m paper_2510_00932_b200.timeline`
 * turns the stamps into a timeline of one launch inside a train of launches. */
int stream_dot_timeline_f64(const double *x, const double *y, double *out, size_t n, streamops_stream_t stream,
                            unsigned long long *stamps, unsigned *blocks);
#define STREAMOPS_TIMELINE_MAX_BLOCKS 1024

/* Dot without any allocation (the paper has no counterpart; this entry point exists for callers
 * that cannot allocate device memory when they need the result: code that runs after a memory
 * pool has taken the whole device, loops that must not take the allocator's lock or trigger its
 * implicit synchronisation, hosts whose rule is that libraries do not allocate).
 * Same contract as stream_dot_f64 -- device pointers, asynchronous on `stream`, out[0] receives the
 * fp64 dot product, same fixed-order summation so repeated calls give identical bits, same
 * accuracy -- with these differences:
 *   - The partial sums live in a fixed 33,024-byte array inside the library image instead of the
 *     allocated workspace. Every GPU that loads the library holds that array until the process
 *     exits. The call path runs no cudaMalloc, cudaFree or allocating library routine, and does
 *     not create the workspace of streamops_init.
 *   - n may not exceed STREAMOPS_DOT_NOALLOC_MAX_N (2^28 elements, 2 GiB per input): each partial
 *     sum covers a fixed span of 65,536 elements and the array holds 4,096 of them. Larger n
 *     returns STREAMOPS_ERR_TOO_LARGE and launches nothing.
 *   - One array per device, shared by every call and every stream, keeping the previous call's
 *     contents (the entry point re-zeroes the part that must start at zero). Two calls that
 *     overlap in time on one GPU race on it and give wrong results: keep them on one stream or
 *     order them with events.
 *   - The first call on each device looks up the array's device address (once, with that device
 *     current) and is the first launch from this part of the library, which makes the CUDA runtime
 *     load the module that holds the kernel and the array: the driver reserves device memory for
 *     them at that moment. So make one call per device at start-up -- outside stream capture, and
 *     before the device's memory is handed to a pool that takes all of it; n = 1 is enough. Calls
 *     after that first one leave the amount of free device memory unchanged.
 * The summation order differs from stream_dot_f64's, so the two agree to rounding, not bitwise. */
int stream_dot_noalloc_f64(const double *x, const double *y, double *out, double scalar, size_t n, streamops_stream_t stream);
#define STREAMOPS_DOT_NOALLOC_MAX_N (1ull << 28)

/* One pass of the five kernels over three DEVICE arrays of n elements each, in the textbook
 * STREAM dataflow: c <- a; b <- s*c; c <- a+b; a <- b+s*c; dot_out[0] <- dot(a, b). Exactly the five
 * stream_* calls above issued back to back on `stream` (asynchronous, nothing synchronised), from
 * one library call: at L2-resident sizes -- the paper's ARRAY_SIZE values, Table 1 -- the host's
 * per-call cost is what limits an iteration, and the edits the paper reports for these kernels
 * (Table 2) were all on that side. The sequence can be captured into a CUDA graph (call
 * streamops_init first: capture must not allocate). a, b, c must be distinct arrays. */
int streamops_chain_f64(double *a, double *b, double *c, double *dot_out, double scalar, size_t n, streamops_stream_t stream);
int streamops_chain_f32(float *a, float *b, float *c, float *dot_out, double scalar, size_t n, streamops_stream_t stream);

/* One pass of the five kernels over three HOST arrays of n elements each, in the textbook
 * STREAM dataflow: c <- a; b <- s*c; c <- a+b; a <- b+s*c; dot(a, b). On return a, b and c hold the results;
 * of their contents on entry only a's are read (the dataflow overwrites c and b before reading them, so b and c
 * are outputs only and are not copied to the device: one array goes up, three come down). The arrays are cut
 * into pieces of 16 MiB per array; each piece is copied into a ring of four device stages (three piece buffers
 * each: 192 MiB of device memory whatever n is, so the arrays may be far larger than the device's
 * memory), run through the five kernels and copied back on three streams of the library's own, so
 * that uploads, kernels and downloads of different pieces overlap and both directions of the host
 * link are in use at once; the call returns after all results are in host memory. The dot product is the left-to-right sum of the pieces' double-
 * precision partial dot products, rounded once: a fixed function of n, repeatable bit for bit, and
 * within the same tolerance as stream_dot_* (not bitwise equal to it). a, b, c and dot_out are HOST
 * pointers owned by the caller (pinned memory lets the copies overlap; pageable memory works).
 * The ring is allocated on the first call and reused while the piece size does not change;
 * streamops_shutdown frees it. Calls from several threads on one device are serialised while they
 * issue their work and wait only for their own results. This is the end-to-end entry point for
 * callers whose data lives on the host. */
int streamops_chain_host_f64(double *a, double *b, double *c, double scalar, size_t n, double *dot_out);
int streamops_chain_host_f32(float *a, float *b, float *c, double scalar, size_t n, float *dot_out);
/* Size of one piece of the host-buffer pipeline, per array, in MiB (1..4096; default 16). The dot
 * product's last bits depend on it (the pieces' partial sums are folded in order). */
int streamops_set_host_piece_mib(int mib);

/* Shared-memory exchange microkernel. Table 1 of the paper lists a shared-memory benchmark whose one
 * parameter is a repetition count (300..1500, default 600) and whose time goes into shared-memory
 * loads and stores (Table 2); the paper does not define it, so the operation is this library's own:
 *   the n 32-bit words of x are cut into tiles of 8 rows x 1024 columns (row-major, 8192 words);
 *   one round replaces, in every tile, row k by row k + row ((k + 1) mod 8) + row ((k + 2) mod 8),
 *   all eight rows taken from the values before the round, addition modulo 2^32; a word past the
 *   last whole tile is a one-row tile of its own and is tripled by a round; out = the array after
 *   `rounds` rounds.
 * (Equivalently row k of the result is sum_j w_j * row (k + j) mod 8, w_j the sum of the coefficients
 * of x^m, m = j mod 8, in (1 + x + x^2)^rounds. The round is a bijection, so the output depends on
 * every input word and on `rounds` however many rounds are run.) Every round moves
 * each word through shared memory once in each direction: 8 * rounds bytes of shared-memory
 * traffic per word against 8 bytes of global traffic, so for rounds >> 5 the kernel is bound by
 * shared-memory bandwidth (128 bytes per clock per SM).
 * x and out are DEVICE pointers to n words, 4-byte aligned (16-byte alignment of both selects the
 * widest shared-memory accesses), out == x allowed, any other overlap is STREAMOPS_ERR_OVERLAP;
 * asynchronous on `stream`; n == 0 does nothing. streamops_set_shmem_width picks the width of one
 * shared-memory access for A/B runs: 4, 8 or 16 bytes (default 16); the result does not depend on it. */
int shmem_mix_u32(const unsigned *x, unsigned *out, unsigned rounds, size_t n, streamops_stream_t stream);
int streamops_set_shmem_width(int bytes);
int streamops_get_shmem_width(void);

/* Creates the per-device state for `device` (SM count, the Dot workspace: partial sums, arrival
 * tickets, an error flag; a few MiB). Optional: every entry point does it on first use for the
 * current device. Allocates device memory, so call it outside stream capture. */
int streamops_init(int device);

/* Frees every per-device workspace and host-path buffer. The library can be used again after. */
int streamops_shutdown(void);

/* Tuning of one (op, dtype) pair: which kernel family and launch shape the entry point uses.
 * Meant for benchmarking A/B runs; the defaults are the measured best on B200. Results of the
 * elementwise kernels do not depend on it; Dot's summation order (hence its last bits) does. */
typedef struct streamops_tuning {
    int kind;           /* 0 = register-vector kernel (ld/st.global), 1 = bulk-copy (TMA) pipeline */
    int vec_bytes;      /* kind 0: 16 or 32 (256-bit ld/st.global) */
    int unroll;         /* kind 0: vectors per thread per array in flight: 1, 2 or 4 */
    int threads;        /* threads per block: 128, 256 or 512 (kind 1: consumer threads) */
    int blocks_per_sm;  /* persistent grid = blocks_per_sm * SMs; 0 = one block per tile (Dot: 0 = 2 or 3 per
                           SM, chosen from the number of tiles) */
    int policy;         /* kind 0 cache-hint set, 0..8 (see streamops_policy_name) */
    int contiguous;     /* 0 = tiles interleaved across blocks, 1 = one contiguous range per block */
    int chunk_bytes;    /* kind 1: bytes per bulk copy per array (multiple of 16, <= 65536) */
    int stages;         /* kind 1: ring depth, 2..8 */
    int two_pass;       /* Dot only: 1 = second pass as its own launch, 0 = last block finishes */
    int reverse;        /* kind 0: 0 = walk the arrays from start to end, 1 = from end to start, 2 = automatic
                           (elementwise kernels; the default): from the end IF an input of this call is the
                           array the previous elementwise call on this device wrote and that call finished
                           at the high end, so that the lines it left in L2 are read first. Results do not
                           depend on the direction; Dot treats 2 as 0 (its summation order is fixed) */
    int pdl;            /* kind 0: 1 = programmatic dependent launch: the kernel's blocks may become
                           resident while the previous kernel of the stream drains, and wait inside
                           the kernel until it has completed (hides launch latency) */
    int keep_mib;       /* kind 0, policies 7 and 8, in a call one of whose inputs is the array the previous
                           elementwise call on the device wrote (a link of a dataflow chain, whose own output
                           is likely to be read next): the last keep_mib MiB of output in traversal order are
                           stored plainly (7) or with evict_last L2 priority (8) and are what the kernel
                           leaves in L2 for its consumer; everything before is stored evict_first, so that
                           the kernel's own output does not push out the lines its producer left there. In
                           any other call policies 7 and 8 store evict_first throughout, as policy 4 */
    int compensated;    /* Dot, kind 0: 1 = carry every accumulator as a (sum, error) pair (two-sum and, for
                           double inputs, an exact product split: the published Dot2 scheme): the result is
                           as accurate as a sum done in about twice the working precision, for inputs whose
                           dot product cancels heavily; ~10 double operations per element instead of one */
    int pipeline;       /* Dot, kind 0, 32-byte vectors: 1 = rolling-slot kernel: a thread keeps `unroll` (2 or 4)
                           slots of one vector per array, folds the oldest into its accumulator and reloads it
                           at once, so that loads stay in flight all the time; 0 = a tile of `unroll` vectors per
                           array is requested, awaited and folded as a whole */
} streamops_tuning_t;

int streamops_set_tuning(int op, int dtype, const streamops_tuning_t *t);
int streamops_get_tuning(int op, int dtype, streamops_tuning_t *t);
int streamops_reset_tuning(void);
const char *streamops_policy_name(int policy);

/* Reads the device error flag of the current device (a bounded wait that gave up sets it),
 * after synchronising `stream`. Returns STREAMOPS_OK or STREAMOPS_ERR_TIMEOUT and clears it. */
int streamops_check(streamops_stream_t stream);

/* Number of attempts a wait on an mbarrier inside the bulk-copy pipelines (tuning kind 1) makes
 * before it gives up; 0 restores the default, 2^22 (seconds). The first attempt is a probe that
 * never blocks, later ones may each suspend the thread for a hardware-defined time. Exists so that
 * the give-up path can be exercised: with a limit of 1 a wait gives up at once unless its data is
 * already there, the kernel sets the error flag, lets the copies it has in flight land (that wait
 * keeps the full limit) and returns, and streamops_check reports STREAMOPS_ERR_TIMEOUT once. The
 * output of such a launch is incomplete. Nothing faults and nothing waits without bound. */
int streamops_set_wait_limit(unsigned tries);

/* Index checking (debugging builds only: the library built with -DSTREAMOPS_CHECK_INDICES, which
 * `python -m paper_2510_00932_b200.build --checked` writes to libstreamops_checked.so). In such a build every
 * global-memory access of the register-vector elementwise and Dot kernels is first checked against the
 * length of its array; an access that does not fit is not made, and the first one is recorded.
 * streamops_index_violation synchronises the device and returns 1 if an access was refused since the last
 * call (filling in which access -- 1/2/3 elementwise load of x / load of y / store, 4 elementwise ragged end,
 * 5/6/7 the same for Dot, 99 the self-test --, its byte offset and the array's byte length, and clearing
 * the record), 0 if none was, and a negative value in a build without checking (-STREAMOPS_ERR_ARG) or on a
 * CUDA error. streamops_index_selftest launches a kernel that only ASKS the checker about an access of
 * `width` bytes at byte `offset` of an array of `limit` bytes, and about the last access that fits, without
 * touching memory: it returns bit 0 = the first was accepted, bit 1 = the second was (so 2 for an `offset`
 * that does not fit, after which streamops_index_violation reports where = 99), negative as above. */
int streamops_index_violation(int *where, unsigned long long *offset, unsigned long long *limit);
int streamops_index_selftest(unsigned long long offset, unsigned long long width, unsigned long long limit);

const char *streamops_status_string(int status);
int streamops_last_cuda_error(void); /* the cudaError_t behind the last STREAMOPS_ERR_CUDA */

/* Number of kernels this library has launched since it was loaded (all devices, all threads). */
unsigned long long streamops_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* STREAMOPS_H */
