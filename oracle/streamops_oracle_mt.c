/*
 * All-cores form of the CPU oracle -- TEST INFRASTRUCTURE, used only to report how long the
 * oracle takes on every host core. It adds no arithmetic of its own: the index range is cut
 * into `nthreads` contiguous pieces and each piece is handed to the single-thread oracle
 * function. The elementwise kernels are independent per index, so their output is identical to
 * the single-thread run. For Dot the per-piece (sum, error) pairs are combined in piece order
 * with the same error-free two-term sum the oracle uses, so the result does not depend on
 * thread timing.
 */
#include <pthread.h>
#include <stddef.h>

void oracle_copy_f64(const double *, double *, size_t);
void oracle_copy_f32(const float *, float *, size_t);
void oracle_scale_f64(const double *, double *, double, size_t);
void oracle_scale_f32(const float *, float *, double, size_t);
void oracle_add_f64(const double *, const double *, double *, size_t);
void oracle_add_f32(const float *, const float *, float *, size_t);
void oracle_triad_f64(const double *, const double *, double *, double, size_t);
void oracle_triad_f32(const float *, const float *, float *, double, size_t);
void oracle_dot2_pair_f64(const double *, const double *, size_t, double *, double *);
void oracle_dot_neumaier_pair_f32(const float *, const float *, size_t, double *, double *);

enum { OP_COPY = 0, OP_SCALE = 1, OP_ADD = 2, OP_TRIAD = 3, OP_DOT = 4 };
#define ORACLE_MAX_THREADS 1024

struct piece {
    int op, is_f64;
    const void *x, *y;
    void *out;
    double scalar;
    size_t begin, count;
    double pair[2];
};

static void *run_piece(void *arg)
{
    struct piece *p = arg;
    const size_t b = p->begin, n = p->count;
    if (p->is_f64) {
        const double *x = (const double *)p->x + b;
        const double *y = p->y ? (const double *)p->y + b : NULL;
        double *out = p->out ? (double *)p->out + b : NULL;
        switch (p->op) {
        case OP_COPY:  oracle_copy_f64(x, out, n); break;
        case OP_SCALE: oracle_scale_f64(x, out, p->scalar, n); break;
        case OP_ADD:   oracle_add_f64(x, y, out, n); break;
        case OP_TRIAD: oracle_triad_f64(x, y, out, p->scalar, n); break;
        case OP_DOT:   oracle_dot2_pair_f64(x, y, n, &p->pair[0], &p->pair[1]); break;
        }
    } else {
        const float *x = (const float *)p->x + b;
        const float *y = p->y ? (const float *)p->y + b : NULL;
        float *out = p->out ? (float *)p->out + b : NULL;
        switch (p->op) {
        case OP_COPY:  oracle_copy_f32(x, out, n); break;
        case OP_SCALE: oracle_scale_f32(x, out, p->scalar, n); break;
        case OP_ADD:   oracle_add_f32(x, y, out, n); break;
        case OP_TRIAD: oracle_triad_f32(x, y, out, p->scalar, n); break;
        case OP_DOT:   oracle_dot_neumaier_pair_f32(x, y, n, &p->pair[0], &p->pair[1]); break;
        }
    }
    return NULL;
}

/* Runs op over [0, n) on nthreads threads. For OP_DOT the result is stored to *dot_out
 * (a double for both precisions) and `out` is ignored. Returns 0, or -1 on a bad argument or
 * a thread that could not be started. */
int oracle_run_mt(int op, int is_f64, const void *x, const void *y, void *out, double scalar,
                  size_t n, int nthreads, double *dot_out)
{
    static struct piece pieces[ORACLE_MAX_THREADS];
    pthread_t tid[ORACLE_MAX_THREADS];
    if (nthreads < 1 || nthreads > ORACLE_MAX_THREADS || op < OP_COPY || op > OP_DOT)
        return -1;
    const size_t base = n / (size_t)nthreads, extra = n % (size_t)nthreads;
    size_t begin = 0;
    int started = 0, rc = 0;
    for (int t = 0; t < nthreads; ++t) {
        struct piece *p = &pieces[t];
        p->op = op; p->is_f64 = is_f64; p->x = x; p->y = y; p->out = out; p->scalar = scalar;
        p->begin = begin;
        p->count = base + ((size_t)t < extra ? 1 : 0);
        p->pair[0] = p->pair[1] = 0.0;
        begin += p->count;
        if (pthread_create(&tid[t], NULL, run_piece, p) != 0) { rc = -1; break; }
        ++started;
    }
    for (int t = 0; t < started; ++t)
        pthread_join(tid[t], NULL);
    if (rc != 0)
        return rc;
    if (op == OP_DOT && dot_out) {
        /* combine in piece order: error-free sum of the running sums, plain sum of the errors */
        double P = pieces[0].pair[0], S = pieces[0].pair[1];
        for (int t = 1; t < nthreads; ++t) {
            const double a = P, b = pieces[t].pair[0];
            const double s = a + b;
            const double bv = s - a;
            const double q = (a - (s - bv)) + (b - bv);
            P = s;
            S += q + pieces[t].pair[1];
        }
        *dot_out = P + S;
    }
    return 0;
}
