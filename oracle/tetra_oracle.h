/*
 * Tetra CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, scalar restatement of what the Tetra decode-and-multiply path
 * computes, written from the paper's definitions only.  It shares no code,
 * table, constant generator or helper with the CUDA library, and the CUDA
 * library never calls it.  Only the test-suite, the smoke check and the bench
 * harness's CPU-baseline leg may load it.
 *
 * Paper passages followed (section / equation / figure):
 *   - Leech lattice, integer form ............ Sec. 3.1, Eq. (1)
 *   - shape-gain reconstruction .............. Sec. 3.1, Eq. (2)
 *   - three octads, the 64-state trellis ..... Sec. 3.2, Fig. "geom"
 *   - state bits, rank vectors, cost, cls,
 *     the 4096-row table, the middle list .... Sec. 3.3, Eq. (3)
 *   - the 48-bit word, the six-load decode ... Sec. 3.4, Fig. "decode"
 *   - table sizes, 1/sqrt(16 m) .............. Sec. 3.4 (last paragraph)
 *   - row scale and unquantized tail ......... Sec. 4.1, Sec. 5.1
 *
 * Readings taken where the paper is silent (each is a labelling choice; none
 * changes the properties the paper states):
 *   R1  Golay code = Turyn construction from the two extended cyclic [8,4]
 *       Hamming codes (generators 1+x+x^3 and 1+x^2+x^3); the three bytes of a
 *       codeword are the three octad sections.
 *   R2  Coordinate j of a section is bit j of its pattern byte and nibble j of
 *       its rank row.
 *   R3  A trellis state is labelled by the low six bits of the section byte
 *       whose bit 7 is clear; a state's 16 branches are in ascending order of
 *       the middle byte; prefix/suffix choice bit 1 complements the byte.
 *   R4  Rank lists: the values of o + 4Z in order of |value|, a tie (+2/-2)
 *       taking the positive value first.  Only this order gives the class
 *       property of Sec. 3.3.
 *   R5  Rows are sorted by (cost, packed 32-bit row value ascending).
 *   R6  mix(i) = i for i < N0, else 2048 + (i - N0).
 *   R7  Word fields, least significant bit first:
 *       i1[0..10] i2[11..21] i3[22..32] s8[33..38] b1[39] b2[40..43] b3[44]
 *       p[45] r[46] g[47]; stored as six little-endian bytes.
 *   R8  The tail is added after the row-scale multiply and is not scaled.
 *
 * Pins (see tests/test_oracle_pins.py): Golay weight enumerator, 64 states per
 * cut, 4096 distinct paths, N0 = 1240 / 808, 18,816-byte blob, m <= 26 and
 * max|y| = 10 over the whole codebook, origin -> zeros, class == parity of the
 * k sum for every pattern byte, cost == squared norm when p = 1, codebook
 * size 2^47 with the first Leech theta-series coefficients 196560 and
 * 16773120 on shells m = 2, 3, Eq. (1) membership and pairwise inner products
 * = 0 mod 8 of decoded points, injectivity on sub-cubes, matvec against a
 * generic dense product.
 */
#ifndef TETRA_ORACLE_H
#define TETRA_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    TO_NCODE = 4096,       /* |G24| */
    TO_NROWS = 4096,       /* rank rows, class 0 then class 1 */
    TO_HALF = 2048,        /* rows per class, and length of the middle list */
    TO_BLOB_BYTES = 18816  /* 16384 + 2304 + 128, Sec. 3.4 */
};

/* All tables the decoder reads, plus the codeword list they were built from. */
typedef struct {
    uint32_t golay[TO_NCODE]; /* codeword: bit 8s+j = coordinate j of section s */
    uint8_t prefixes[128];    /* [2*s8 + b1]  -> pattern byte of section 1 */
    uint16_t branches[1024];  /* [16*s8 + b2] -> byte of section 2 | s16 << 8 */
    uint8_t suffixes[128];    /* [2*s16 + b3] -> pattern byte of section 3 */
    uint32_t rows[TO_NROWS];  /* rank rows, 4 bits per rank, nibble j = coord j */
    int32_t n0;               /* class-0 rows among the 2048 cheapest overall */
    int8_t val[4][8];         /* val[o][rho] = to_rank_value(o, rho), filled at build */
} to_tables;

/* Build every table from first principles.  Returns 0, or a negative code if
 * a structural count the paper states does not hold (never expected). */
int to_build_tables(to_tables *t);

/* cost(rho) and cls(rho) of a packed rank row, Sec. 3.3. */
int to_row_cost(uint32_t row);
int to_row_cls(uint32_t row);

/* The rho-th value of o + 4Z counted outward from zero (o in 0..3, rho in 0..7). */
int to_rank_value(int o, int rho);

/* Row index the middle section reads, and its class delta, Sec. 3.3. */
int to_mix(const to_tables *t, int i2, int *delta);

/* One section: parity p, pattern byte c, rank row -> eight coordinates. */
void to_decode_section(const to_tables *t, int p, int cbyte, uint32_t row, int8_t y8[8]);

/* One 48-bit word -> 24 coordinates, shell index m = sum(y^2)/16, gain bit g. */
void to_decode_word(const to_tables *t, uint64_t word, int8_t y[24], int *m, int *g);

/* n words of 6 little-endian bytes each -> y[n][24], m[n], g[n]. */
void to_decode_blocks(const to_tables *t, const uint8_t *codes, size_t n,
                      int8_t *y, uint8_t *m, uint8_t *g);

/* Eq. (1) membership test, independent of the decoder: 1 if y is in the lattice. */
int to_in_leech(const to_tables *t, const int8_t y[24]);

/* The paper's table blob: rows (u32 LE) | prefixes | branches (u16 LE) |
 * suffixes | 32 floats 1/sqrt(16 m) with entry 0 = 0 (double, rounded once). */
void to_table_blob(const to_tables *t, uint8_t blob[TO_BLOB_BYTES]);

/*
 * FP64 matrix-vector product with decoded weights, Eq. (2) + Sec. 5.1:
 *   out[n] = sigma[n] * sum_b gain[g_nb]/sqrt(16 m_nb) * sum_j Y_nbj x[24 b + j]
 *            + sum_t tail[n][t] * x[24 B + t]
 * codes:  N rows of `row_stride` bytes, block b of a row at byte 6 b.
 * x:      doubles, length >= 24*B + ntail (caller zero-extends for zero-padding).
 * tail:   N x ntail doubles or NULL (ntail = 0).
 * out:    N doubles.  termnorm (optional): sqrt(sum_k (sigma w x)^2) per row.
 * abssum (optional): sum_k |sigma w x| per row.  threads <= 1: serial.
 * Returns the number of threads used.
 */
int to_gemv(const to_tables *t, const uint8_t *codes, size_t row_stride,
            int N, int B, const float *sigma, const float gain[2],
            const double *x, const double *tail, int ntail,
            double *out, double *termnorm, double *abssum, int threads);

#ifdef __cplusplus
}
#endif
#endif
