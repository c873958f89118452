/* CPU oracle for the 4-bit group-quantised matrices -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * Plain, slow, FP64.  It restates what the paper says about its other weight
 * format: an int4 record holds 4-bit weights in groups of 128 along a row with a
 * float16 scale and a float16 offset per group (Sec. 4.1); the embedding table
 * and the output head use the same record with groups of 64 (Sec. 4.4); the
 * kernel dequantises each weight with its group's scale and offset and
 * accumulates the products (Sec. 5.1); embedding rows are dequantised on the
 * fly for the input tokens (Sec. 4.4).
 *
 * Readings where the paper leaves a choice (the same ones the CUDA library
 * documents in its header):
 *   Q1  a weight is  w = scale * q + offset  with q in 0..15 unsigned;
 *   Q2  byte b of a row holds weight 2b in its low nibble, 2b+1 in its high nibble;
 *   Q3  scale and offset are stored as [row][group], group = k / G;
 *   Q4  K must be a multiple of G (every shape of the three models is);
 *   Q5  a dequantised embedding row is float16: fma(scale, q, offset) rounded once
 *       to float32, then rounded to nearest-even float16.
 *
 * Pins (tests/test_q4_oracle_pins.py): the half conversions against numpy for
 * every bit pattern; single-nibble matrices (nibble order, row/column order);
 * offset-only and scale-ramp matrices with closed-form results (group
 * boundaries); the dense product of numpy on matrices unpacked by numpy.
 *
 * Nothing here is shared with the CUDA path; only tests, the smoke check and the
 * bench harness's CPU legs may use it. */
#ifndef Q4_ORACLE_H
#define Q4_ORACLE_H
#include <stddef.h>
#include <stdint.h>

double q4o_half_to_double(uint16_t h);
uint16_t q4o_float_to_half(float f);

/* Exact value of weight (n, k) as a double (Q1-Q3). */
double q4o_weight(const uint8_t *q, const uint16_t *scale, const uint16_t *offset, int K, int G, size_t n, int k);

/* y[v][n] = sum_k w(n,k) * x[v][k] in FP64; termnorm[v][n] = sqrt(sum_k (w x)^2) if not NULL.
 * Returns 0, or -1 on a bad size. */
int q4o_gemv(const uint8_t *q, const uint16_t *scale, const uint16_t *offset, const uint16_t *x, int N, int K,
             int G, int batch, double *y, double *termnorm, int threads);

/* out[t][k] = float16 of row ids[t] (Q5).  Returns 0, -1 on a bad size, -2 on an id out of range. */
int q4o_rows(const uint8_t *q, const uint16_t *scale, const uint16_t *offset, const int32_t *ids, int count, int N,
             int K, int G, uint16_t *out);
#endif
