/*
 * CPU oracle for the five streaming kernels -- TEST INFRASTRUCTURE, not part of the product.
 *
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may call this file.
 * It shares no code, header, table or constant with the CUDA library.
 *
 * The paper (Table 1 and Section 5.2) names the kernels -- Copy, Mul, Add, Triad, Dot, taken from
 * a STREAM-style benchmark -- without printing a formula, so each function below is the textbook
 * definition of the named vector operation, written as the plainest possible scalar loop:
 *
 *   Copy   out[i] = x[i]                       (bit for bit)
 *   Mul    out[i] = RN(s * x[i])               ("scale")
 *   Add    out[i] = RN(x[i] + y[i])
 *   Triad  out[i] = RN(x[i] + RN(s * y[i]))    (two roundings, never a fused multiply-add)
 *   Dot    sum_i x[i] * y[i]                   (an accuracy reference: compensated summation)
 *
 * RN is IEEE-754 round-to-nearest-even in the array's own precision; the scalar arrives as a
 * double and is rounded once to that precision before the loop.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math (contraction off so that a*b+c never
 * becomes an FMA; no value-changing optimisation). x86-64 SSE arithmetic: no excess precision.
 *
 * Pins (tests, CPU only): exact rational arithmetic on random and crafted operands for the four
 * elementwise kernels; exact big-integer dot products, closed forms, unit vectors, cancellation
 * patterns and a long-double cross-check for Dot. No function here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

/* ------------------------------------------------------------------ Copy (Table 1, "Copy") */

void oracle_copy_f64(const double *x, double *out, size_t n)
{
    for (size_t i = 0; i < n; ++i) {
        uint64_t bits;                      /* move the bit pattern, so NaN payloads survive */
        memcpy(&bits, &x[i], sizeof bits);
        memcpy(&out[i], &bits, sizeof bits);
    }
}

void oracle_copy_f32(const float *x, float *out, size_t n)
{
    for (size_t i = 0; i < n; ++i) {
        uint32_t bits;
        memcpy(&bits, &x[i], sizeof bits);
        memcpy(&out[i], &bits, sizeof bits);
    }
}

/* ------------------------------------------------------------------ Mul / scale (Table 1, "Mul") */

void oracle_scale_f64(const double *x, double *out, double scalar, size_t n)
{
    for (size_t i = 0; i < n; ++i)
        out[i] = scalar * x[i];
}

void oracle_scale_f32(const float *x, float *out, double scalar, size_t n)
{
    const float s = (float)scalar;          /* one rounding of the scalar, before the loop */
    for (size_t i = 0; i < n; ++i)
        out[i] = s * x[i];
}

/* ------------------------------------------------------------------ Add (Table 1, "Add") */

void oracle_add_f64(const double *x, const double *y, double *out, size_t n)
{
    for (size_t i = 0; i < n; ++i)
        out[i] = x[i] + y[i];
}

void oracle_add_f32(const float *x, const float *y, float *out, size_t n)
{
    for (size_t i = 0; i < n; ++i)
        out[i] = x[i] + y[i];
}

/* ------------------------------------------------------------------ Triad (Table 1, "Triad") */

void oracle_triad_f64(const double *x, const double *y, double *out, double scalar, size_t n)
{
    for (size_t i = 0; i < n; ++i) {
        const double prod = scalar * y[i];  /* rounded product ... */
        out[i] = x[i] + prod;               /* ... then a rounded sum */
    }
}

void oracle_triad_f32(const float *x, const float *y, float *out, double scalar, size_t n)
{
    const float s = (float)scalar;
    for (size_t i = 0; i < n; ++i) {
        const float prod = s * y[i];
        out[i] = x[i] + prod;
    }
}

/* ------------------------------------------------------------------ Dot (Table 1, "Dot")
 *
 * fp64: the compensated dot product "Dot2" of Ogita, Rump and Oishi (Accurate Sum and Dot
 * Product, SIAM J. Sci. Comput. 2005): every product is split without error into its rounded
 * value and its rounding error, the rounded values are accumulated with an error-free two-term
 * sum, and all the error terms are accumulated beside it. The result is as accurate as if the
 * sum had been formed in about twice the working precision and rounded once.
 *
 * The pair form returns the running sum p and the error accumulator s separately so that a
 * caller can combine several ranges in a fixed order; the dot product of the range is p + s.
 */

static void two_sum(double a, double b, double *sum, double *err)
{
    const double t = a + b;
    const double bv = t - a;
    *err = (a - (t - bv)) + (b - bv);
    *sum = t;
}

static void two_prod(double a, double b, double *prod, double *err)
{
    const double p = a * b;
    *err = fma(a, b, -p);                   /* exact: a*b - RN(a*b) is representable */
    *prod = p;
}

void oracle_dot2_pair_f64(const double *x, const double *y, size_t n, double *p_out, double *s_out)
{
    double p = 0.0, s = 0.0;
    if (n > 0)
        two_prod(x[0], y[0], &p, &s);
    for (size_t i = 1; i < n; ++i) {
        double h, r, q;
        two_prod(x[i], y[i], &h, &r);
        two_sum(p, h, &p, &q);
        s += (q + r);
    }
    *p_out = p;
    *s_out = s;
}

double oracle_dot_f64(const double *x, const double *y, size_t n)
{
    double p, s;
    oracle_dot2_pair_f64(x, y, n, &p, &s);
    return p + s;
}

/* Cross-check for the above, by a different route: each product's two exact halves are summed
 * in long double (64-bit significand) with Neumaier's compensated summation. */
double oracle_dot_f64_longdouble(const double *x, const double *y, size_t n)
{
    long double sum = 0.0L, comp = 0.0L;
    for (size_t i = 0; i < n; ++i) {
        double h, r;
        two_prod(x[i], y[i], &h, &r);
        const long double terms[2] = { (long double)h, (long double)r };
        for (int k = 0; k < 2; ++k) {
            const long double v = terms[k];
            const long double t = sum + v;
            if (fabsl(sum) >= fabsl(v))
                comp += (sum - t) + v;
            else
                comp += (v - t) + sum;
            sum = t;
        }
    }
    return (double)(sum + comp);
}

/* fp32 inputs: the product of two floats has at most 48 significant bits, so it is exact in
 * double; the exact products are summed in double with Neumaier's compensated summation.
 * Returned in double (callers compare before and after rounding to float). */
void oracle_dot_neumaier_pair_f32(const float *x, const float *y, size_t n, double *sum_out, double *comp_out)
{
    double sum = 0.0, comp = 0.0;
    for (size_t i = 0; i < n; ++i) {
        const double v = (double)x[i] * (double)y[i];
        const double t = sum + v;
        if (fabs(sum) >= fabs(v))
            comp += (sum - t) + v;
        else
            comp += (v - t) + sum;
        sum = t;
    }
    *sum_out = sum;
    *comp_out = comp;
}

double oracle_dot_f32(const float *x, const float *y, size_t n)
{
    double sum, comp;
    oracle_dot_neumaier_pair_f32(x, y, n, &sum, &comp);
    return sum + comp;
}

/* Sum of |x[i]*y[i]|: the denominator of the relative-error test when the dot product itself is
 * zero, and the numerator of the condition number. Plain long-double accumulation. */
double oracle_dot_abs_f64(const double *x, const double *y, size_t n)
{
    long double acc = 0.0L;
    for (size_t i = 0; i < n; ++i)
        acc += fabsl((long double)x[i] * (long double)y[i]);
    return (double)acc;
}

double oracle_dot_abs_f32(const float *x, const float *y, size_t n)
{
    long double acc = 0.0L;
    for (size_t i = 0; i < n; ++i)
        acc += fabsl((long double)x[i] * (long double)y[i]);
    return (double)acc;
}

/* Fold of per-GPU partial sums (the exchange step of a Dot over an array split across GPUs):
 * the doubles added strictly left to right, one rounding per addition; the caller rounds the
 * total to the element type. */
double oracle_fold_f64(const double *p, size_t count)
{
    double acc = 0.0;
    for (size_t i = 0; i < count; ++i)
        acc = acc + p[i];
    return acc;
}
