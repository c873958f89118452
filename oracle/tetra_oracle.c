/*
 * Tetra CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.  See tetra_oracle.h.
 *
 * Everything here is the definition written out: codewords are enumerated,
 * trellis tables are found by searching the codeword list, rank rows are
 * enumerated and sorted, a word is decoded one field and one coordinate at a
 * time, and the product is three nested loops in double.
 */
#include "tetra_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* Golay code (Sec. 3.2; reading R1)                                   */
/* ------------------------------------------------------------------ */

static int bit_parity(unsigned v)
{
    int par = 0;
    while (v) {
        par ^= (int)(v & 1u);
        v >>= 1;
    }
    return par;
}

/* The 16 words of the extended cyclic [8,4] code whose generator polynomial
 * has coefficient bits `gen` (bit i = coefficient of x^i, degree 3): all
 * combinations of gen, x gen, x^2 gen, x^3 gen, each with an overall parity
 * bit appended as bit 7. */
static void extended_hamming(unsigned gen, uint8_t out[16])
{
    for (unsigned msg = 0; msg < 16; ++msg) {
        unsigned w = 0;
        for (int i = 0; i < 4; ++i)
            if (msg & (1u << i))
                w ^= gen << i;
        w |= (unsigned)bit_parity(w) << 7;
        out[msg] = (uint8_t)w;
    }
}

static int cmp_u32(const void *a, const void *b)
{
    uint32_t x = *(const uint32_t *)a, y = *(const uint32_t *)b;
    return (x > y) - (x < y);
}

/* Turyn: (a+x | b+x | a+b+x), a, b in H, x in H'.  Section s is byte s. */
static int build_golay(uint32_t code[TO_NCODE])
{
    uint8_t h[16], hr[16];
    extended_hamming(0x0Bu, h);  /* 1 + x + x^3   */
    extended_hamming(0x0Du, hr); /* 1 + x^2 + x^3 */
    int n = 0;
    for (int a = 0; a < 16; ++a)
        for (int b = 0; b < 16; ++b)
            for (int x = 0; x < 16; ++x) {
                uint32_t c1 = (uint32_t)(h[a] ^ hr[x]);
                uint32_t c2 = (uint32_t)(h[b] ^ hr[x]);
                uint32_t c3 = (uint32_t)(h[a] ^ h[b] ^ hr[x]);
                code[n++] = c1 | (c2 << 8) | (c3 << 16);
            }
    qsort(code, TO_NCODE, sizeof(uint32_t), cmp_u32);
    for (int i = 1; i < TO_NCODE; ++i)
        if (code[i] == code[i - 1])
            return -1; /* not 4096 distinct words */
    return 0;
}

static int in_golay(const uint32_t code[TO_NCODE], uint32_t w)
{
    return bsearch(&w, code, TO_NCODE, sizeof(uint32_t), cmp_u32) != NULL;
}

/* ------------------------------------------------------------------ */
/* Trellis tables (Sec. 3.2, Fig. "geom"; reading R3)                  */
/* ------------------------------------------------------------------ */

/* The section byte with bit 7 clear that carries state label s: its low seven
 * bits have even weight, so bit 6 is the parity of the low six. */
static unsigned state_byte(unsigned s)
{
    return s | ((unsigned)bit_parity(s) << 6);
}

static int build_trellis(to_tables *t)
{
    for (unsigned s = 0; s < 64; ++s) {
        t->prefixes[2 * s + 0] = (uint8_t)state_byte(s);
        t->prefixes[2 * s + 1] = (uint8_t)(state_byte(s) ^ 0xFFu);
        t->suffixes[2 * s + 0] = (uint8_t)state_byte(s);
        t->suffixes[2 * s + 1] = (uint8_t)(state_byte(s) ^ 0xFFu);
    }
    for (unsigned s = 0; s < 64; ++s) {
        unsigned c1 = state_byte(s);
        int nbranch = 0;
        for (unsigned c2 = 0; c2 < 256; ++c2) {        /* ascending middle byte */
            for (unsigned c3 = 0; c3 < 128; ++c3) {     /* the suffix with bit 7 clear */
                if (!in_golay(t->golay, c1 | (c2 << 8) | (c3 << 16)))
                    continue;
                if (c3 != state_byte(c3 & 63u))
                    return -2; /* suffix is not of the labelled form */
                if (nbranch >= 16)
                    return -3; /* more than 16 branches out of a state */
                t->branches[16 * s + nbranch] = (uint16_t)(c2 | ((c3 & 63u) << 8));
                ++nbranch;
            }
        }
        if (nbranch != 16)
            return -4;
    }
    /* 64 * 2 * 16 * 2 paths must spell out the code exactly once each. */
    static uint8_t seen[1u << 24];
    memset(seen, 0, sizeof seen);
    for (unsigned s = 0; s < 64; ++s)
        for (unsigned b1 = 0; b1 < 2; ++b1)
            for (unsigned b2 = 0; b2 < 16; ++b2)
                for (unsigned b3 = 0; b3 < 2; ++b3) {
                    unsigned c1 = t->prefixes[2 * s + b1];
                    unsigned br = t->branches[16 * s + b2];
                    unsigned c3 = t->suffixes[2 * (br >> 8) + b3];
                    uint32_t w = c1 | ((br & 0xFFu) << 8) | (c3 << 16);
                    if (!in_golay(t->golay, w) || seen[w])
                        return -5;
                    seen[w] = 1;
                }
    return 0;
}

/* ------------------------------------------------------------------ */
/* Rank rows (Sec. 3.3; readings R2, R5, R6)                           */
/* ------------------------------------------------------------------ */

int to_row_cost(uint32_t row)
{
    int cost = 0;
    for (int j = 0; j < 8; ++j) {
        int rho = (int)((row >> (4 * j)) & 15u);
        cost += (2 * rho + 1) * (2 * rho + 1);
    }
    return cost;
}

int to_row_cls(uint32_t row)
{
    int cls = 0;
    for (int j = 0; j < 8; ++j) {
        int rho = (int)((row >> (4 * j)) & 15u);
        if (rho == 1 || rho == 2 || rho == 5 || rho == 6)
            cls ^= 1;
    }
    return cls;
}

typedef struct {
    int cost;
    uint32_t row;
} ranked_row;

static int cmp_ranked(const void *a, const void *b)
{
    const ranked_row *x = (const ranked_row *)a, *y = (const ranked_row *)b;
    if (x->cost != y->cost)
        return (x->cost > y->cost) - (x->cost < y->cost);
    return (x->row > y->row) - (x->row < y->row);
}

/* Append every rank vector in {0..7}^8 with cost <= bound. */
static void enum_rows(int coord, uint32_t partial, int cost, int bound,
                      ranked_row *out, size_t *n, size_t cap)
{
    if (coord == 8) {
        if (*n < cap) {
            out[*n].cost = cost;
            out[*n].row = partial;
        }
        ++*n;
        return;
    }
    for (int rho = 0; rho < 8; ++rho) {
        int c = cost + (2 * rho + 1) * (2 * rho + 1);
        if (c + (7 - coord) > bound) /* every later coordinate costs at least 1 */
            break;
        enum_rows(coord + 1, partial | ((uint32_t)rho << (4 * coord)), c, bound,
                  out, n, cap);
    }
}

static int build_rows(to_tables *t)
{
    /* Raise the cost bound until both classes hold at least 2048 vectors; the
     * list is then complete below the bound, so its cheapest 2048 per class
     * are the cheapest overall. */
    const size_t cap = (size_t)1 << 22;
    ranked_row *all = (ranked_row *)malloc(cap * sizeof *all);
    if (!all)
        return -10;
    size_t n = 0;
    for (int bound = 8;; bound += 8) {
        n = 0;
        enum_rows(0, 0, 0, bound, all, &n, cap);
        if (n > cap) {
            free(all);
            return -11;
        }
        size_t count[2] = {0, 0};
        for (size_t i = 0; i < n; ++i)
            ++count[to_row_cls(all[i].row)];
        if (count[0] >= TO_HALF && count[1] >= TO_HALF)
            break;
    }
    qsort(all, n, sizeof *all, cmp_ranked);

    int filled[2] = {0, 0};
    for (size_t i = 0; i < n; ++i) {
        int cls = to_row_cls(all[i].row);
        if (filled[cls] < TO_HALF) {
            t->rows[TO_HALF * cls + filled[cls]] = all[i].row;
            ++filled[cls];
        }
    }
    /* The middle list: the 2048 cheapest of both classes together. */
    int n0 = 0;
    for (size_t i = 0; i < TO_HALF; ++i)
        if (to_row_cls(all[i].row) == 0)
            ++n0;
    t->n0 = n0;
    free(all);
    return 0;
}

int to_mix(const to_tables *t, int i2, int *delta)
{
    if (i2 < t->n0) {
        if (delta)
            *delta = 0;
        return i2;
    }
    if (delta)
        *delta = 1;
    return TO_HALF + (i2 - t->n0);
}

int to_build_tables(to_tables *t)
{
    memset(t, 0, sizeof *t);
    int rc = build_golay(t->golay);
    if (rc)
        return rc;
    rc = build_trellis(t);
    if (rc)
        return rc;
    for (int o = 0; o < 4; ++o)
        for (int rho = 0; rho < 8; ++rho)
            t->val[o][rho] = (int8_t)to_rank_value(o, rho);
    return build_rows(t);
}

/* ------------------------------------------------------------------ */
/* Decode (Sec. 3.3, Sec. 3.4, Fig. "decode"; readings R4, R7)         */
/* ------------------------------------------------------------------ */

int to_rank_value(int o, int rho)
{
    /* Candidates o + 4 t around zero, ordered by |value|, positive first on a
     * tie; the answer is entry rho of that list. */
    int cand[33], n = 0;
    for (int tt = -16; tt <= 16; ++tt)
        cand[n++] = o + 4 * tt;
    for (int i = 1; i < n; ++i) { /* insertion sort */
        int v = cand[i], k = i - 1;
        while (k >= 0 && (abs(cand[k]) > abs(v) ||
                          (abs(cand[k]) == abs(v) && cand[k] < v))) {
            cand[k + 1] = cand[k];
            --k;
        }
        cand[k + 1] = v;
    }
    return cand[rho];
}

void to_decode_section(const to_tables *t, int p, int cbyte, uint32_t row, int8_t y8[8])
{
    for (int j = 0; j < 8; ++j) {
        int cj = (cbyte >> j) & 1;
        int o = p + 2 * cj;
        int rho = (int)((row >> (4 * j)) & 15u);
        y8[j] = t->val[o][rho & 7]; /* the rho-th value of o + 4Z */
    }
}

void to_decode_word(const to_tables *t, uint64_t word, int8_t y[24], int *m, int *g)
{
    int i1 = (int)(word & 0x7FFu);
    int i2 = (int)((word >> 11) & 0x7FFu);
    int i3 = (int)((word >> 22) & 0x7FFu);
    int s8 = (int)((word >> 33) & 0x3Fu);
    int b1 = (int)((word >> 39) & 1u);
    int b2 = (int)((word >> 40) & 0xFu);
    int b3 = (int)((word >> 44) & 1u);
    int p = (int)((word >> 45) & 1u);
    int r = (int)((word >> 46) & 1u);
    int gg = (int)((word >> 47) & 1u);

    /* trellis reads: the suffix waits for the state the branch returns */
    int c1 = t->prefixes[2 * s8 + b1];
    int br = t->branches[16 * s8 + b2];
    int c2 = br & 0xFF;
    int s16 = br >> 8;
    int c3 = t->suffixes[2 * s16 + b3];

    /* row reads */
    int delta;
    uint32_t row1 = t->rows[TO_HALF * r + i1];
    uint32_t row2 = t->rows[to_mix(t, i2, &delta)];
    int r3 = p ^ r ^ delta; /* Eq. (3) */
    uint32_t row3 = t->rows[TO_HALF * r3 + i3];

    to_decode_section(t, p, c1, row1, y);
    to_decode_section(t, p, c2, row2, y + 8);
    to_decode_section(t, p, c3, row3, y + 16);

    int norm = 0;
    for (int j = 0; j < 24; ++j)
        norm += y[j] * y[j];
    if (m)
        *m = norm / 16;
    if (g)
        *g = gg;
}

void to_decode_blocks(const to_tables *t, const uint8_t *codes, size_t n,
                      int8_t *y, uint8_t *m, uint8_t *g)
{
    for (size_t i = 0; i < n; ++i) {
        uint64_t w = 0;
        for (int k = 0; k < 6; ++k)
            w |= (uint64_t)codes[6 * i + k] << (8 * k);
        int mm, gg;
        to_decode_word(t, w, y + 24 * i, &mm, &gg);
        if (m)
            m[i] = (uint8_t)mm;
        if (g)
            g[i] = (uint8_t)gg;
    }
}

/* ------------------------------------------------------------------ */
/* Lattice membership, Eq. (1), written without the decoder            */
/* ------------------------------------------------------------------ */

int to_in_leech(const to_tables *t, const int8_t y[24])
{
    int p = y[0] & 1;
    uint32_t c = 0;
    int ksum = 0;
    for (int j = 0; j < 24; ++j) {
        int v = y[j];
        if ((v & 1) != p)
            return 0;
        int half = (v - p) / 2; /* exact: v - p is even */
        int cj = half & 1;      /* two's complement: correct for negatives */
        int rest = v - p - 2 * cj;
        if (rest % 4 != 0)
            return 0;
        ksum += rest / 4;
        c |= (uint32_t)cj << j;
    }
    if (!in_golay(t->golay, c))
        return 0;
    return (ksum & 1) == p;
}

/* ------------------------------------------------------------------ */
/* Table blob (Sec. 3.4, last paragraph)                               */
/* ------------------------------------------------------------------ */

void to_table_blob(const to_tables *t, uint8_t blob[TO_BLOB_BYTES])
{
    size_t off = 0;
    for (int i = 0; i < TO_NROWS; ++i)
        for (int k = 0; k < 4; ++k)
            blob[off++] = (uint8_t)(t->rows[i] >> (8 * k));
    memcpy(blob + off, t->prefixes, 128);
    off += 128;
    for (int i = 0; i < 1024; ++i) {
        blob[off++] = (uint8_t)(t->branches[i] & 0xFF);
        blob[off++] = (uint8_t)(t->branches[i] >> 8);
    }
    memcpy(blob + off, t->suffixes, 128);
    off += 128;
    for (int mm = 0; mm < 32; ++mm) {
        float f = mm ? (float)(1.0 / sqrt(16.0 * (double)mm)) : 0.0f;
        uint32_t u;
        memcpy(&u, &f, 4);
        for (int k = 0; k < 4; ++k)
            blob[off++] = (uint8_t)(u >> (8 * k));
    }
}

/* ------------------------------------------------------------------ */
/* FP64 product (Eq. (2), Sec. 5.1; reading R8)                        */
/* ------------------------------------------------------------------ */

static void gemv_row(const to_tables *t, const uint8_t *row_codes, int B,
                     double sigma, const float gain[2], const double *x,
                     const double *tail, int ntail,
                     double *out, double *termnorm, double *abssum)
{
    double acc = 0.0, sq = 0.0, ab = 0.0;
    for (int b = 0; b < B; ++b) {
        uint64_t w = 0;
        for (int k = 0; k < 6; ++k)
            w |= (uint64_t)row_codes[6 * b + k] << (8 * k);
        int8_t y[24];
        int m, g;
        to_decode_word(t, w, y, &m, &g);
        double scale = m ? (double)gain[g] / sqrt(16.0 * (double)m) : 0.0;
        double dot = 0.0;
        for (int j = 0; j < 24; ++j) {
            double term = (double)y[j] * x[24 * b + j];
            dot += term;
            double wx = sigma * scale * term;
            sq += wx * wx;
            ab += fabs(wx);
        }
        acc += scale * dot;
    }
    double res = sigma * acc;
    for (int tt = 0; tt < ntail; ++tt) {
        double wx = tail[tt] * x[24 * B + tt];
        res += wx;
        sq += wx * wx;
        ab += fabs(wx);
    }
    *out = res;
    if (termnorm)
        *termnorm = sqrt(sq);
    if (abssum)
        *abssum = ab;
}

int to_gemv(const to_tables *t, const uint8_t *codes, size_t row_stride,
            int N, int B, const float *sigma, const float gain[2],
            const double *x, const double *tail, int ntail,
            double *out, double *termnorm, double *abssum, int threads)
{
    int used = 1;
#ifdef _OPENMP
    if (threads > 1)
        used = threads;
#pragma omp parallel for schedule(static) num_threads(used)
#else
    (void)threads;
#endif
    for (int n = 0; n < N; ++n)
        gemv_row(t, codes + (size_t)n * row_stride, B, (double)sigma[n], gain, x,
                 tail ? tail + (size_t)n * (size_t)ntail : NULL, ntail,
                 out + n, termnorm ? termnorm + n : NULL, abssum ? abssum + n : NULL);
    return used;
}
