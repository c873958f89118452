// Host-side table construction for the Tetra library.
//
// Written from the paper's statements alone and on a different route from the
// test oracle's: the Golay code comes from a 12 x 24 generator matrix, the
// trellis tables are filled by scattering every codeword into the slot its own
// bytes name (Sec. 3.2), and the rank rows are enumerated in base 5 and split
// by class before sorting (Sec. 3.3).
#include "tetra_tables.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

namespace tetra {
namespace {

inline int parity8(unsigned v) { return __builtin_popcount(v & 0xFFu) & 1; }

// Basis of the extended cyclic [8,4] code with generator polynomial bits `gen`.
void hamming_basis(unsigned gen, uint8_t basis[4]) {
    for (int i = 0; i < 4; ++i) {
        unsigned w = (gen << i) & 0x7Fu;
        basis[i] = static_cast<uint8_t>(w | (parity8(w) << 7));
    }
}

inline uint8_t span4(const uint8_t basis[4], unsigned msg) {
    uint8_t w = 0;
    for (int i = 0; i < 4; ++i)
        if (msg & (1u << i)) w ^= basis[i];
    return w;
}

// Turyn construction: codeword bytes (h(a)+h'(x), h(b)+h'(x), h(a)+h(b)+h'(x)).
struct Turyn {
    uint8_t h[4], hr[4];
    Turyn() {
        hamming_basis(0x0Bu, h);   // 1 + x + x^3
        hamming_basis(0x0Du, hr);  // 1 + x^2 + x^3
    }
    void bytes(unsigned a, unsigned b, unsigned x, uint8_t c[3]) const {
        const uint8_t ha = span4(h, a), hb = span4(h, b), hx = span4(hr, x);
        c[0] = ha ^ hx;
        c[1] = hb ^ hx;
        c[2] = ha ^ hb ^ hx;
    }
};

// State label of a section byte: its low six bits once bit 7 is cleared by
// complementing; the choice bit is the original bit 7.
inline void state_of(uint8_t c, unsigned* state, unsigned* choice) {
    *choice = c >> 7;
    *state = (*choice ? static_cast<uint8_t>(~c) : c) & 63u;
}

int build_trellis(const Turyn& t, PaperTables* p, uint16_t abx_of[4096]) {
    // Scatter pass 1: which middle bytes leave each state, and where they lead.
    int16_t next_state[64][256];
    for (auto& row : next_state) std::fill(std::begin(row), std::end(row), int16_t(-1));
    bool have_prefix[128] = {}, have_suffix[128] = {};
    for (unsigned a = 0; a < 16; ++a)
        for (unsigned b = 0; b < 16; ++b)
            for (unsigned x = 0; x < 16; ++x) {
                uint8_t c[3];
                t.bytes(a, b, x, c);
                unsigned s8, b1, s16, b3;
                state_of(c[0], &s8, &b1);
                state_of(c[2], &s16, &b3);
                p->prefixes[2 * s8 + b1] = c[0];
                p->suffixes[2 * s16 + b3] = c[2];
                have_prefix[2 * s8 + b1] = have_suffix[2 * s16 + b3] = true;
                if (next_state[s8][c[1]] >= 0 && next_state[s8][c[1]] != int(s16)) return -1;
                next_state[s8][c[1]] = static_cast<int16_t>(s16);
            }
    for (int i = 0; i < 128; ++i)
        if (!have_prefix[i] || !have_suffix[i]) return -2;
    // A state's branches in ascending order of the middle byte.
    uint8_t branch_index[64][256];
    for (unsigned s8 = 0; s8 < 64; ++s8) {
        int n = 0;
        for (unsigned c2 = 0; c2 < 256; ++c2) {
            if (next_state[s8][c2] < 0) continue;
            if (n == 16) return -3;
            p->branches[16 * s8 + n] = static_cast<uint16_t>(c2 | (unsigned(next_state[s8][c2]) << 8));
            branch_index[s8][c2] = static_cast<uint8_t>(n++);
        }
        if (n != 16) return -4;
    }
    // Scatter pass 2: the Turyn coordinates of every trellis path (for the packer).
    std::vector<int> hits(4096, 0);
    for (unsigned a = 0; a < 16; ++a)
        for (unsigned b = 0; b < 16; ++b)
            for (unsigned x = 0; x < 16; ++x) {
                uint8_t c[3];
                t.bytes(a, b, x, c);
                unsigned s8, b1, s16, b3;
                state_of(c[0], &s8, &b1);
                state_of(c[2], &s16, &b3);
                const unsigned path = s8 | (b1 << 6) | (unsigned(branch_index[s8][c[1]]) << 7) | (b3 << 11);
                abx_of[path] = static_cast<uint16_t>(a | (b << 4) | (x << 8));
                ++hits[path];
            }
    for (int h : hits)
        if (h != 1) return -5;  // 64 * 2 * 16 * 2 paths, one per codeword
    return 0;
}

inline int row_cost(uint32_t row) {
    int c = 0;
    for (int j = 0; j < 8; ++j) {
        const int r = (row >> (4 * j)) & 15;
        c += (2 * r + 1) * (2 * r + 1);
    }
    return c;
}

inline int row_class(uint32_t row) {
    int k = 0;
    for (int j = 0; j < 8; ++j) {
        const int r = (row >> (4 * j)) & 15;
        k ^= (0x66 >> r) & 1;  // ranks 1, 2, 5, 6
    }
    return k;
}

int build_rows(PaperTables* p, int* n0_out) {
    // Ranks 0..4 suffice: a rank of 5 costs 121 alone, above every kept row
    // (checked below), so base-5 digits enumerate all candidates.
    std::vector<uint64_t> keys[2];  // cost << 32 | row: sorts by cost, then by row value
    for (unsigned code = 0; code < 390625u; ++code) {
        uint32_t row = 0;
        unsigned rest = code;
        for (int j = 0; j < 8; ++j) {
            row |= (rest % 5u) << (4 * j);
            rest /= 5u;
        }
        keys[row_class(row)].push_back((uint64_t(row_cost(row)) << 32) | row);
    }
    for (int cls = 0; cls < 2; ++cls) {
        if (keys[cls].size() < 2048) return -10;
        std::partial_sort(keys[cls].begin(), keys[cls].begin() + 2048, keys[cls].end());
        if ((keys[cls][2047] >> 32) >= 121 + 7) return -11;
        for (int i = 0; i < 2048; ++i) p->rows[2048 * cls + i] = static_cast<uint32_t>(keys[cls][i]);
    }
    // The middle list: merge the two sorted halves and stop after 2048 rows.
    int i0 = 0, i1 = 0;
    while (i0 + i1 < 2048) {
        if (keys[0][i0] < keys[1][i1]) ++i0; else ++i1;
    }
    *n0_out = i0;
    return 0;
}

}  // namespace

int build_device_tables(DeviceTables* out, const float* gain2) {
    std::memset(out, 0, sizeof *out);
    Turyn turyn;
    int rc = build_trellis(turyn, &out->paper, out->trellis_to_abx);
    if (rc) return rc;
    int n0 = 0;
    rc = build_rows(&out->paper, &n0);
    if (rc) return rc;
    if (n0 != kMiddleClass0) return -20;
    out->paper.rsqrt16m[0] = 0.0f;
    for (int m = 1; m < 32; ++m) out->paper.rsqrt16m[m] = static_cast<float>(1.0 / std::sqrt(16.0 * m));
    out->gain[0] = gain2 ? gain2[0] : 4.3156f;
    out->gain[1] = gain2 ? gain2[1] : 5.4415f;
    out->magic = kTableMagic;
    out->version = kTableVersion;

    // Fast-path rows.  Per class: rows holding a rank-4 coordinate go to the first
    // kRank4Slots slots, topped up with rows that use ranks 0 and 1 only (a patched
    // pool serves ranks 0, 1 and 4); everything else keeps its order behind them.
    for (int cls = 0; cls < 2; ++cls) {
        std::vector<int> tail_rows, fillers, front;
        for (int i = 0; i < 2048; ++i) {
            const uint32_t row = out->paper.rows[2048 * cls + i];
            int max_rank = 0, n4 = 0;
            for (int j = 0; j < 8; ++j) {
                const int r = (row >> (4 * j)) & 15;
                if (r > 4) return -21;
                if (r == 4) ++n4;
                if (r > max_rank) max_rank = r;
            }
            if (n4 > 1) return -22;
            if (n4 == 1) {
                for (int j = 0; j < 8; ++j) {  // the other coordinates of such a row are of rank 0 or 1
                    const int r = (row >> (4 * j)) & 15;
                    if (r == 2 || r == 3) return -24;
                }
                tail_rows.push_back(i);
            } else if (max_rank <= 1) {
                fillers.push_back(i);
            } else {
                front.push_back(i);
            }
        }
        if (int(tail_rows.size()) > kRank4Slots) return -25;
        // Fillers are taken cheapest first and go in front of the rank-4 rows, so slot 0 of class 0 is
        // the all-zero row: the all-zero device word then decodes to the origin, which the kernels rely
        // on when they pad.
        const int nfill = kRank4Slots - int(tail_rows.size());
        if (int(fillers.size()) < nfill) return -26;
        std::vector<int> special(fillers.begin(), fillers.begin() + nfill);
        special.insert(special.end(), tail_rows.begin(), tail_rows.end());
        front.insert(front.end(), fillers.begin() + nfill, fillers.end());
        std::sort(front.begin(), front.end());
        if (int(front.size()) != 2048 - kRank4Slots) return -27;
        if (cls == 0 && out->paper.rows[special[0]] != 0u) return -28;
        for (int slot = 0; slot < 2048; ++slot) {
            const int i = slot < kRank4Slots ? special[slot] : front[slot - kRank4Slots];
            const uint32_t row = out->paper.rows[2048 * cls + i];
            uint32_t fast = 0;
            for (int j = 0; j < 8; ++j) {
                unsigned r = (row >> (4 * j)) & 15u;
                if (r == 4) r = 2;
                fast |= (r << 1) << (4 * j);
            }
            out->rows_fast[2048 * cls + slot] = fast;
            out->row_perm[cls][i] = static_cast<uint16_t>(slot);
        }
    }
    // The middle list keeps its own copy in i2 order; its rows never reach rank 4.
    for (int i2 = 0; i2 < 2048; ++i2) {
        const int idx = i2 < n0 ? i2 : 2048 + (i2 - n0);
        const uint32_t row = out->paper.rows[idx];
        uint32_t fast = 0;
        for (int j = 0; j < 8; ++j) {
            const unsigned r = (row >> (4 * j)) & 15u;
            if (r > 3) return -23;
            fast |= (r << 1) << (4 * j);
        }
        out->mid_fast[i2] = fast;
    }
    for (unsigned v = 0; v < 16; ++v) {
        const uint8_t h = span4(turyn.h, v), hr = span4(turyn.hr, v);
        uint32_t mh = 0, mhr = 0;
        for (int j = 0; j < 8; ++j) {
            mh |= uint32_t((h >> j) & 1) << (4 * j);
            mhr |= uint32_t((hr >> j) & 1) << (4 * j);
        }
        out->mask_h[v] = mh;
        out->mask_hr[v] = mhr;
    }
    for (int g = 0; g < 2; ++g)
        for (int m = 0; m < 32; ++m)
            for (int k = 0; k < 4; ++k) out->scale[g][m][k] = 0.f;
    for (int g = 0; g < 2; ++g)
        for (int m = 0; m < 32; ++m) out->scale[0][m][2 * g] = -(out->gain[g] * out->paper.rsqrt16m[m]);
    return 0;
}

}  // namespace tetra
