/* See tetra_encode_oracle.h. */
#include "tetra_encode_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define NQ 39    /* section norms are multiples of 4 up to 152 */
#define NQ2 77   /* sums of two section norms */
#define NEG (-1e300)

/* Best correlation of one section for (pattern byte, class, norm / 4), with the list index that attains it. */
typedef struct {
    double corr[256][2][NQ];
    int arg[256][2][NQ];
} section_table;

/* List entry -> rank row.  Sections 0 and 2 read rows[2048 cls + i]; the middle section reads the merged
 * list, whose class-0 entries are i2 < n0 and class-1 entries i2 >= n0 (Sec. 3.3). */
static int list_length(const to_tables *t, int section, int cls)
{
    if (section != 1)
        return TO_HALF;
    return cls == 0 ? t->n0 : TO_HALF - t->n0;
}

static uint32_t list_row(const to_tables *t, int section, int cls, int i, int *field)
{
    if (section != 1) {
        *field = i;
        return t->rows[TO_HALF * cls + i];
    }
    int i2 = cls == 0 ? i : t->n0 + i, delta;
    uint32_t row = t->rows[to_mix(t, i2, &delta)];
    *field = i2;
    return row;
}

static void fill_section(const to_tables *t, const double *w8, int p, int section, int row_limit,
                         const uint8_t *bytes, int nbytes, section_table *T)
{
    for (int b = 0; b < 256; ++b)
        for (int c = 0; c < 2; ++c)
            for (int q = 0; q < NQ; ++q) {
                T->corr[b][c][q] = NEG;
                T->arg[b][c][q] = -1;
            }
    int done[256] = {0};
    for (int k = 0; k < nbytes; ++k) {
        int cbyte = bytes[k];
        if (done[cbyte])
            continue; /* the trellis tables repeat their pattern bytes */
        done[cbyte] = 1;
        for (int cls = 0; cls < 2; ++cls) {
            int len = list_length(t, section, cls);
            if (len > row_limit)
                len = row_limit;
            for (int i = 0; i < len; ++i) {
                int field;
                uint32_t row = list_row(t, section, cls, i, &field);
                int8_t y8[8];
                to_decode_section(t, p, cbyte, row, y8);
                double corr = 0.0;
                int norm = 0;
                for (int j = 0; j < 8; ++j) {
                    corr += w8[j] * (double)y8[j];
                    norm += y8[j] * y8[j];
                }
                int q = norm / 4;
                if (corr > T->corr[cbyte][cls][q]) {
                    T->corr[cbyte][cls][q] = corr;
                    T->arg[cbyte][cls][q] = field;
                }
            }
        }
    }
}

int to_encode_block(const to_tables *t, const double w[24], int row_limit, uint64_t *word, double *cosine)
{
    if (row_limit < 1 || row_limit > TO_HALF)
        return -1;
    double wn = 0.0;
    for (int j = 0; j < 24; ++j)
        wn += w[j] * w[j];
    wn = sqrt(wn);
    *word = 0;
    *cosine = 0.0;
    if (wn == 0.0)
        return 0; /* E3 */

    section_table *T = malloc(3 * sizeof(section_table));
    /* F1[s8][cls1][q1]; H[s16][cls1 ^ cls2][q12] */
    double (*F1)[2][NQ] = malloc(64 * sizeof(*F1));
    int (*F1b)[2][NQ] = malloc(64 * sizeof(*F1b));
    double (*H)[2][NQ2] = malloc(64 * sizeof(*H));
    int (*Hs8)[2][NQ2] = malloc(64 * sizeof(*Hs8));  /* s8 | b2 << 6 | cls1 << 10 | q1 << 11 */
    double best = NEG;
    uint64_t best_word = 0;

    uint8_t c2bytes[1024];
    for (int i = 0; i < 1024; ++i)
        c2bytes[i] = (uint8_t)(t->branches[i] & 0xFF);

    for (int p = 0; p < 2; ++p) {
        fill_section(t, w, p, 0, row_limit, t->prefixes, 128, &T[0]);
        fill_section(t, w + 8, p, 1, row_limit, c2bytes, 1024, &T[1]);
        fill_section(t, w + 16, p, 2, row_limit, t->suffixes, 128, &T[2]);

        /* first cut: the better of the two prefixes of a state */
        for (int s8 = 0; s8 < 64; ++s8)
            for (int c1 = 0; c1 < 2; ++c1)
                for (int q = 0; q < NQ; ++q) {
                    F1[s8][c1][q] = NEG;
                    F1b[s8][c1][q] = 0;
                    for (int b1 = 0; b1 < 2; ++b1) {
                        double v = T[0].corr[t->prefixes[2 * s8 + b1]][c1][q];
                        if (v > F1[s8][c1][q]) {
                            F1[s8][c1][q] = v;
                            F1b[s8][c1][q] = b1;
                        }
                    }
                }
        /* second cut: state after the branch, class parity so far, summed norm */
        for (int s = 0; s < 64; ++s)
            for (int c = 0; c < 2; ++c)
                for (int q = 0; q < NQ2; ++q) {
                    H[s][c][q] = NEG;
                    Hs8[s][c][q] = -1;
                }
        for (int s8 = 0; s8 < 64; ++s8)
            for (int b2 = 0; b2 < 16; ++b2) {
                int br = t->branches[16 * s8 + b2], c2 = br & 0xFF, s16 = br >> 8;
                for (int cls1 = 0; cls1 < 2; ++cls1)
                    for (int q1 = 0; q1 < NQ; ++q1) {
                        double a = F1[s8][cls1][q1];
                        if (a <= NEG)
                            continue;
                        for (int cls2 = 0; cls2 < 2; ++cls2)
                            for (int q2 = 0; q2 < NQ; ++q2) {
                                double b = T[1].corr[c2][cls2][q2];
                                if (b <= NEG)
                                    continue;
                                if (a + b > H[s16][cls1 ^ cls2][q1 + q2]) {
                                    H[s16][cls1 ^ cls2][q1 + q2] = a + b;
                                    Hs8[s16][cls1 ^ cls2][q1 + q2] =
                                        s8 | (b2 << 6) | (cls1 << 10) | (q1 << 11) | (q2 << 17);
                                }
                            }
                    }
            }
        /* last section and the objective */
        for (int s16 = 0; s16 < 64; ++s16)
            for (int b3 = 0; b3 < 2; ++b3) {
                int c3 = t->suffixes[2 * s16 + b3];
                for (int par = 0; par < 2; ++par) {
                    int cls3 = p ^ par; /* Eq. (3): r3 = p ^ r ^ delta */
                    for (int q12 = 0; q12 < NQ2; ++q12) {
                        double a = H[s16][par][q12];
                        if (a <= NEG)
                            continue;
                        for (int q3 = 0; q3 < NQ; ++q3) {
                            double b = T[2].corr[c3][cls3][q3];
                            if (b <= NEG || q12 + q3 == 0)
                                continue;
                            double val = (a + b) / sqrt(4.0 * (double)(q12 + q3));
                            if (val > best) {
                                best = val;
                                int back = Hs8[s16][par][q12];
                                int s8 = back & 63, b2 = (back >> 6) & 15, cls1 = (back >> 10) & 1;
                                int q1 = (back >> 11) & 63, q2 = (back >> 17) & 63;
                                int cls2 = par ^ cls1;
                                int b1 = F1b[s8][cls1][q1];
                                int i1 = T[0].arg[t->prefixes[2 * s8 + b1]][cls1][q1];
                                int i2 = T[1].arg[t->branches[16 * s8 + b2] & 0xFF][cls2][q2];
                                int i3 = T[2].arg[c3][cls3][q3];
                                best_word = (uint64_t)i1 | ((uint64_t)i2 << 11) | ((uint64_t)i3 << 22) |
                                            ((uint64_t)s8 << 33) | ((uint64_t)b1 << 39) | ((uint64_t)b2 << 40) |
                                            ((uint64_t)b3 << 44) | ((uint64_t)p << 45) | ((uint64_t)cls1 << 46);
                            }
                        }
                    }
                }
            }
    }
    free(T);
    free(F1);
    free(F1b);
    free(H);
    free(Hs8);
    *word = best_word;
    *cosine = best / wn;
    return 0;
}

int to_choose_gain(double c, double sigma, const double gain[2])
{
    double e0 = gain[0] * sigma * gain[0] * sigma - 2.0 * gain[0] * sigma * c;
    double e1 = gain[1] * sigma * gain[1] * sigma - 2.0 * gain[1] * sigma * c;
    return e1 < e0 ? 1 : 0;
}

int to_encode_blocks(const to_tables *t, const double *w, size_t n, int row_limit, double sigma,
                     const double gain[2], uint64_t *words, double *cosines, int threads)
{
    if (row_limit < 1 || row_limit > TO_HALF)
        return -1;
#ifdef _OPENMP
    if (threads > 0)
        omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel for schedule(dynamic, 4)
    for (long long i = 0; i < (long long)n; ++i) {
        uint64_t word;
        double cs;
        to_encode_block(t, w + 24 * i, row_limit, &word, &cs);
        double wn = 0.0;
        for (int j = 0; j < 24; ++j)
            wn += w[24 * i + j] * w[24 * i + j];
        int g = to_choose_gain(cs * sqrt(wn), sigma, gain);
        words[i] = word | ((uint64_t)g << 47);
        cosines[i] = cs;
    }
    return 0;
}
