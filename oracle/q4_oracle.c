/* See q4_oracle.h.  Every function is the definition written out. */
#include "q4_oracle.h"

#include <math.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* IEEE 754 binary16 -> double: sign, 5 exponent bits (bias 15), 10 fraction bits. */
double q4o_half_to_double(uint16_t h) {
    const int sign = (h >> 15) & 1, e = (h >> 10) & 31, f = h & 1023;
    double v;
    if (e == 0)
        v = ldexp((double)f, -24); /* zero and subnormals: f * 2^-24 */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexp((double)(1024 + f), e - 25); /* (1 + f/1024) * 2^(e-15) */
    return sign ? -v : v;
}

/* float -> binary16, round to nearest, ties to even, by exact arithmetic on the value. */
uint16_t q4o_float_to_half(float f) {
    const uint16_t sign = signbit(f) ? 0x8000u : 0u;
    double a = fabs((double)f);
    if (isnan(f)) return (uint16_t)(sign | 0x7E00u);
    if (a == 0.0) return sign;
    if (isinf(f)) return (uint16_t)(sign | 0x7C00u);
    int ex;
    (void)frexp(a, &ex); /* a = m * 2^ex, 0.5 <= m < 1, so a is in [2^(ex-1), 2^ex) */
    int e = ex - 1;      /* a in [2^e, 2^(e+1)) */
    if (e < -14) e = -14; /* subnormal range shares the spacing of the smallest normal binade */
    /* spacing of representable values in this binade is 2^(e-10) */
    const double units = ldexp(a, 10 - e); /* exact: a power-of-two scaling */
    double r = nearbyint(units);           /* default rounding mode: nearest, ties to even */
    long long n = (long long)r;            /* value = n * 2^(e-10), n <= 2048 */
    if (n >= 2048) {                       /* rounded up into the next binade */
        n = 1024;
        e += 1;
    }
    if (e > 15) return (uint16_t)(sign | 0x7C00u); /* overflow to infinity */
    if (n < 1024) return (uint16_t)(sign | (uint16_t)n); /* subnormal (e == -14) or zero */
    return (uint16_t)(sign | (uint16_t)((e + 15) << 10) | (uint16_t)(n - 1024));
}

static int nibble(const uint8_t *q, int K, size_t n, int k) {
    const uint8_t b = q[n * (size_t)(K / 2) + (size_t)(k / 2)];
    return (k & 1) ? (b >> 4) : (b & 15);
}

double q4o_weight(const uint8_t *q, const uint16_t *scale, const uint16_t *offset, int K, int G, size_t n, int k) {
    const size_t groups = (size_t)(K / G), g = (size_t)(k / G);
    return q4o_half_to_double(scale[n * groups + g]) * (double)nibble(q, K, n, k) +
           q4o_half_to_double(offset[n * groups + g]);
}

int q4o_gemv(const uint8_t *q, const uint16_t *scale, const uint16_t *offset, const uint16_t *x, int N, int K,
             int G, int batch, double *y, double *termnorm, int threads) {
    if (N < 0 || K <= 0 || G <= 0 || K % G || K % 2 || batch < 1) return -1;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel for schedule(static)
    for (long long n = 0; n < N; ++n)
        for (int v = 0; v < batch; ++v) {
            double s = 0.0, t2 = 0.0;
            for (int k = 0; k < K; ++k) {
                const double term = q4o_weight(q, scale, offset, K, G, (size_t)n, k) *
                                    q4o_half_to_double(x[(size_t)v * K + k]);
                s += term;
                t2 += term * term;
            }
            y[(size_t)v * N + n] = s;
            if (termnorm) termnorm[(size_t)v * N + n] = sqrt(t2);
        }
    return 0;
}

int q4o_rows(const uint8_t *q, const uint16_t *scale, const uint16_t *offset, const int32_t *ids, int count, int N,
             int K, int G, uint16_t *out) {
    if (N < 0 || K <= 0 || G <= 0 || K % G || K % 2 || count < 0) return -1;
    for (int t = 0; t < count; ++t) {
        if (ids[t] < 0 || ids[t] >= N) return -2;
        for (int k = 0; k < K; ++k) {
            /* scale*q + offset is exact in double (15 + 11 significant bits, exponents within 40 of each
             * other); one rounding to float32 (Q5), then one to float16 */
            const float w32 = (float)q4o_weight(q, scale, offset, K, G, (size_t)ids[t], k);
            out[(size_t)t * K + k] = q4o_float_to_half(w32);
        }
    }
    return 0;
}
