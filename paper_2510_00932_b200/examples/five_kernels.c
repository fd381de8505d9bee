/*
 * The five streaming kernels (Table 1 of the paper: Copy, Mul, Add, Triad, Dot) called from plain C
 * through libstreamops' C ABI: device memory from the CUDA runtime, no Python, no torch.
 *
 *   gcc -O2 -I include -I /usr/local/cuda/include paper_2510_00932_b200/examples/five_kernels.c \
 *       -L paper_2510_00932_b200 -lstreamops -L /usr/local/cuda/lib64 -lcudart \
 *       -Wl,-rpath,$PWD/paper_2510_00932_b200 -o five_kernels && ./five_kernels [n]
 *
 * Runs one pass c <- a; b <- s*c; c <- a+b; a <- b+s*c; dot(a, b) on constant arrays, for which every
 * result has a closed form (with a = 1, b = 2, c = 0, s = 0.5: c = 1, b = 0.5, c = 1.5, a = 1.25,
 * dot = n * 1.25 * 0.5, all exact in binary floating point), checks them, and prints GB/s per kernel.
 */
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>

#include "streamops.h"

#define CUDA_OK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { \
    fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_)); return 2; } } while (0)
#define STREAM_OK(call) do { int s_ = (call); if (s_ != STREAMOPS_OK) { \
    fprintf(stderr, "%s: %s\n", #call, streamops_status_string(s_)); return 3; } } while (0)

static int all_equal(const double *v, size_t n, double want) {
    for (size_t i = 0; i < n; ++i) if (v[i] != want) return 0;
    return 1;
}

int main(int argc, char **argv) {
    const size_t n = argc > 1 ? (size_t)atoll(argv[1]) : ((size_t)1 << 24) + 5;
    const double s = 0.5;
    double *a, *b, *c, *d, *host = (double *)malloc(n * sizeof(double)), dot = 0.0;
    if (!host) return 1;
    CUDA_OK(cudaMalloc((void **)&a, n * sizeof(double)));
    CUDA_OK(cudaMalloc((void **)&b, n * sizeof(double)));
    CUDA_OK(cudaMalloc((void **)&c, n * sizeof(double)));
    CUDA_OK(cudaMalloc((void **)&d, sizeof(double)));
    for (size_t i = 0; i < n; ++i) host[i] = 1.0;
    CUDA_OK(cudaMemcpy(a, host, n * sizeof(double), cudaMemcpyHostToDevice));
    for (size_t i = 0; i < n; ++i) host[i] = 2.0;
    CUDA_OK(cudaMemcpy(b, host, n * sizeof(double), cudaMemcpyHostToDevice));
    CUDA_OK(cudaMemset(c, 0, n * sizeof(double)));
    cudaStream_t stream;
    CUDA_OK(cudaStreamCreate(&stream));
    STREAM_OK(streamops_init(0));

    /* one checked pass */
    STREAM_OK(stream_copy_f64(a, c, 0.0, n, stream));
    STREAM_OK(stream_scale_f64(c, b, s, n, stream));
    STREAM_OK(stream_add_f64(a, b, c, 0.0, n, stream));
    STREAM_OK(stream_triad_f64(b, c, a, s, n, stream));
    STREAM_OK(stream_dot_f64(a, b, d, 0.0, n, stream));
    STREAM_OK(streamops_check(stream));                  /* synchronises; reports a kernel wait that gave up */
    CUDA_OK(cudaMemcpy(&dot, d, sizeof(double), cudaMemcpyDeviceToHost));
    int ok = dot == (double)n * 1.25 * 0.5;
    CUDA_OK(cudaMemcpy(host, a, n * sizeof(double), cudaMemcpyDeviceToHost)); ok &= all_equal(host, n, 1.25);
    CUDA_OK(cudaMemcpy(host, b, n * sizeof(double), cudaMemcpyDeviceToHost)); ok &= all_equal(host, n, 0.5);
    CUDA_OK(cudaMemcpy(host, c, n * sizeof(double), cudaMemcpyDeviceToHost)); ok &= all_equal(host, n, 1.5);
    if (!ok) { fprintf(stderr, "results differ from the closed forms (dot %.17g)\n", dot); return 4; }

    /* timing: each kernel 20 times in a row (a is rewritten by triad: values change, the timing does not) */
    cudaEvent_t e0, e1;
    CUDA_OK(cudaEventCreate(&e0)); CUDA_OK(cudaEventCreate(&e1));
    const char *names[5] = {"copy", "scale", "add", "triad", "dot"};
    const double arrays[5] = {2, 2, 3, 3, 2};
    for (int op = 0; op < 5; ++op) {
        float ms = 0.f;
        for (int rep = 0; rep < 23; ++rep) {
            if (rep == 3) CUDA_OK(cudaEventRecord(e0, stream));
            switch (op) {
                case 0: STREAM_OK(stream_copy_f64(a, c, 0.0, n, stream)); break;
                case 1: STREAM_OK(stream_scale_f64(c, b, s, n, stream)); break;
                case 2: STREAM_OK(stream_add_f64(a, b, c, 0.0, n, stream)); break;
                case 3: STREAM_OK(stream_triad_f64(b, c, a, s, n, stream)); break;
                default: STREAM_OK(stream_dot_f64(a, b, d, 0.0, n, stream)); break;
            }
        }
        CUDA_OK(cudaEventRecord(e1, stream));
        CUDA_OK(cudaEventSynchronize(e1));
        CUDA_OK(cudaEventElapsedTime(&ms, e0, e1));
        printf("%-5s %8.2f us  %8.1f GB/s\n", names[op], ms / 20 * 1e3, arrays[op] * n * 8 / (ms / 20 * 1e-3) / 1e9);
    }
    printf("ok: n = %zu, dot = %.17g, %llu kernels launched\n", n, dot, streamops_launch_count());
    STREAM_OK(streamops_shutdown());
    cudaFree(a); cudaFree(b); cudaFree(c); cudaFree(d); free(host);
    return 0;
}
