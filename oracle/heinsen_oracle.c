/*
 * heinsen_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, sequential float64 CPU evaluation of the first-order linear
 * recurrence
 *
 *        x_t = a_t * x_{t-1} + b_t ,   t = 1..n ,   x_0 given
 *
 * (Abstract; Summary, first two paragraphs; Proof, first sentence), for
 * `rows` independent sequences stored row-major.  The paper's two-prefix-sum
 * expression (Eq. 1-3, Eq. 7-8) reaches exactly this sequence in real
 * arithmetic (Proof, Eq. 4-6), so the definition itself is the oracle: one
 * element at a time, no blocking, no reordering, nothing shared with the CUDA
 * path.  The only parallelism is OpenMP over independent rows.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may load
 * this file.  The product path never does.
 *
 * Storage types (`dtype`): 0 = IEEE float32, 1 = bfloat16 (upper 16 bits of a
 * float32), 2 = float64.  Stored values are widened exactly to float64 before
 * any arithmetic; outputs are always float64.
 *
 * Pinned by tests/test_oracle_pins.py (closed forms, rational brute force of
 * Eq. 4, Eq. 7 restated with library scans, invariants).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double widen(const void *p, int64_t i, int dtype) {
    if (dtype == 0) return (double)((const float *)p)[i];
    if (dtype == 1) {
        uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return ((const double *)p)[i];
}

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Linear domain.  x[r,t-1] = a[r,t-1]*x_prev + b[r,t-1] with x_prev = x0[r]
 * at t = 1 (Abstract; Proof, Eq. 4 first line).  n outputs per row; x_0 is
 * not part of the output (Eq. 7's tail()).  Signed inputs need nothing
 * special: the reals are closed under the two operations (Summary, last
 * paragraph).
 */
void oracle_scan_linear(const void *a, const void *b, const void *x0, double *x,
                        int64_t rows, int64_t n, int dtype, int nthreads) {
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double xp = widen(x0, r, dtype);
        for (int64_t t = 0; t < n; ++t) {
            const int64_t i = r * n + t;
            xp = widen(a, i, dtype) * xp + widen(b, i, dtype);
            x[i] = xp;
        }
    }
}

/* log(e^p + sigma * e^q) for p >= q, sigma = +1 (same sign) or -1 (opposite). */
static inline double log_sum_or_diff(double p, double q, int opposite) {
    const double d = q - p; /* <= 0 */
    if (!opposite) return p + log1p(exp(d));
    if (d == 0.0) return -INFINITY;
    /* log(1 - e^d): pick the better-conditioned of the two textbook forms. */
    return p + (d > -0.6931471805599453 ? log(-expm1(d)) : log1p(-exp(d)));
}

/*
 * Log domain, sign + magnitude.  The same recurrence, still one element at a
 * time, but carried as (log|x|, sign x) so that magnitudes far outside the
 * float64 range (log b = 800, a* = -2500) cannot overflow:
 *
 *     log|a_t x_{t-1}| = log|a_t| + log|x_{t-1}|,  sign = sign a_t XOR sign x_{t-1}
 *     x_t = (a_t x_{t-1}) + b_t   as a signed log-add.
 *
 * A negative number's logarithm is log|.| + i*pi on the principal branch
 * (Summary, last paragraph: interim logarithms in C, results in R); the
 * imaginary part is carried here as one sign bit, 1 = negative.
 * log 0 = -inf is a legal input.  An exact zero result has sign 0 ('+').
 *
 * sign_a, sign_b: [rows,n] uint8 or NULL (all positive); sign_x0: [rows] or
 * NULL.  sign_x may be NULL when no sign output is wanted.
 */
void oracle_scan_log(const void *log_a, const void *log_b, const void *log_x0,
                     const uint8_t *sign_a, const uint8_t *sign_b, const uint8_t *sign_x0,
                     double *log_x, uint8_t *sign_x,
                     int64_t rows, int64_t n, int dtype, int nthreads) {
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double L = widen(log_x0, r, dtype);
        int s = sign_x0 ? (sign_x0[r] & 1) : 0;
        if (L == -INFINITY) s = 0;
        for (int64_t t = 0; t < n; ++t) {
            const int64_t i = r * n + t;
            /* a_t * x_{t-1} */
            double P = widen(log_a, i, dtype) + L;
            int sp = s ^ (sign_a ? (sign_a[i] & 1) : 0);
            /* + b_t */
            const double Q = widen(log_b, i, dtype);
            const int sq = sign_b ? (sign_b[i] & 1) : 0;
            if (P == -INFINITY) {
                L = Q;
                s = sq;
            } else if (Q == -INFINITY) {
                L = P;
                s = sp;
            } else if (P >= Q) {
                L = log_sum_or_diff(P, Q, sp != sq);
                s = sp;
            } else {
                L = log_sum_or_diff(Q, P, sp != sq);
                s = sq;
            }
            if (L == -INFINITY) s = 0;
            log_x[i] = L;
            if (sign_x) sign_x[i] = (uint8_t)s;
        }
    }
}
