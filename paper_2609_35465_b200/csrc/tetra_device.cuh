// Device-side decoders for Tetra words (sm_100a).
//
// Two decoders live here:
//   * decode_file_word: the six-load decode of Sec. 3.4 (Fig. "decode") on a
//     word in file order, reading the paper-format tables.  Used by
//     tetra_decode_blocks and by the paper-design GEMV.
//   * the fast decoder: works on the re-ordered 48-bit device word written by
//     tetra_pack_codes and on tables staged in shared memory.  It produces the
//     p = 0 image y0 of the lattice point as packed int8 (four coordinates per
//     register, one PRMT per four); the true point is y0 when p = 0 and
//     1 - y0 when p = 1 (shifting o = p + 2c by one maps every rank list of
//     Sec. 3.3 onto one minus the list two places on).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "tetra_tables.h"

namespace tetra {

// ---------------------------------------------------------------------------
// small wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ int dp4a_ss(uint32_t a, uint32_t b, int c) {  // signed a . signed b
    int d;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ int dp4a_su(uint32_t a, uint32_t b, int c) {  // signed a . unsigned b
    int d;
    asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// Loads from the staged tables: they never change after staging, so the loads
// are not volatile and the compiler may schedule them freely.
__device__ __forceinline__ uint32_t lds32(uint32_t saddr) {
    uint32_t v;
    asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(saddr));
    return v;
}
__device__ __forceinline__ float lds32f(uint32_t saddr) {
    float v;
    asm("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(saddr));
    return v;
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------------------
// File-order decode (Sec. 3.3, 3.4)
// ---------------------------------------------------------------------------

// The rho-th element of o + 4Z counted outward from zero, in closed form:
// v0 = 0, 4, -4, 8, -8, ... is the o = 0 list; the other lists are 1 - v0,
// 2 - v0 and v0 - 1.
__device__ __forceinline__ int rank_value(int o, int rho) {
    const int t = (rho + 1) >> 1;
    const int v0 = (rho & 1) ? 4 * t : -4 * t;
    return o == 0 ? v0 : (o == 1 ? 1 - v0 : (o == 2 ? 2 - v0 : v0 - 1));
}

__device__ __forceinline__ uint64_t load_file_word(const uint8_t* codes, size_t block) {
    const uint16_t* p = reinterpret_cast<const uint16_t*>(codes + 6 * block);
    return uint64_t(p[0]) | (uint64_t(p[1]) << 16) | (uint64_t(p[2]) << 32);
}

// T may point to global or shared memory.
__device__ __forceinline__ void decode_file_word(const PaperTables* T, uint64_t w, int y[24], int* m, int* g) {
    const int i1 = int(w & 0x7FF), i2 = int((w >> 11) & 0x7FF), i3 = int((w >> 22) & 0x7FF);
    const int s8 = int((w >> 33) & 63), b1 = int((w >> 39) & 1), b2 = int((w >> 40) & 15), b3 = int((w >> 44) & 1);
    const int p = int((w >> 45) & 1), r = int((w >> 46) & 1);
    *g = int((w >> 47) & 1);
    // trellis: the suffix read waits for the state returned by the branch read
    const int c1 = T->prefixes[2 * s8 + b1];
    const int br = T->branches[16 * s8 + b2];
    const int c3 = T->suffixes[2 * (br >> 8) + b3];
    const int c[3] = {c1, br & 0xFF, c3};
    // rank rows
    const int delta = i2 >= kMiddleClass0;
    const int r3 = p ^ r ^ delta;  // Eq. (3)
    const uint32_t row[3] = {T->rows[2048 * r + i1],
                             T->rows[delta ? 2048 + (i2 - kMiddleClass0) : i2],
                             T->rows[2048 * r3 + i3]};
    int norm = 0;
#pragma unroll
    for (int s = 0; s < 3; ++s)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int o = p + 2 * ((c[s] >> j) & 1);
            const int v = rank_value(o, int((row[s] >> (4 * j)) & 15u));
            y[8 * s + j] = v;
            norm += v * v;
        }
    *m = norm >> 4;
}

// ---------------------------------------------------------------------------
// Device word (written by the pack kernel).  48 bits = w0 (32) + w1 (16):
//   w0: [0..10] i1  [11] r  [12..22] i3  [23] q = p^r  [24..27] a  [28..31] b
//   w1: [0..10] i2  [11..14] x  [15] g
// (a, b, x) are the Turyn coordinates of the trellis path: the three pattern
// bytes are h(a)+h'(x), h(b)+h'(x), h(a)+h(b)+h'(x).
// ---------------------------------------------------------------------------
__device__ __forceinline__ void file_to_device_word(uint64_t w, const uint16_t* trellis_to_abx,
                                                    uint32_t* w0, uint32_t* w1) {
    const uint32_t i1 = uint32_t(w & 0x7FF), i2 = uint32_t((w >> 11) & 0x7FF), i3 = uint32_t((w >> 22) & 0x7FF);
    const uint32_t path = uint32_t((w >> 33) & 0xFFF);
    const uint32_t p = uint32_t((w >> 45) & 1), r = uint32_t((w >> 46) & 1), g = uint32_t((w >> 47) & 1);
    const uint32_t abx = trellis_to_abx[path];
    *w0 = i1 | (r << 11) | (i3 << 12) | ((p ^ r) << 23) | ((abx & 0xFFu) << 24);
    *w1 = i2 | ((abx >> 8) << 11) | (g << 15);
}

// Byte offsets of the staged tables inside the shared-memory copy of the fast part.
constexpr uint32_t kSmRows = 0;
constexpr uint32_t kSmMid = 16384;
constexpr uint32_t kSmScale = 24576;
constexpr uint32_t kSmMaskH = 24832;
constexpr uint32_t kSmMaskHr = 24896;
constexpr uint32_t kSmAlign = 16384;  // the staged copy starts on a 16 KiB boundary of shared memory
static_assert(kSmMid == offsetof(DeviceTables, mid_fast) - kFastOffset, "staged layout");
static_assert(kSmScale == offsetof(DeviceTables, scale) - kFastOffset, "staged layout");
static_assert(kSmMaskH == offsetof(DeviceTables, mask_h) - kFastOffset, "staged layout");
static_assert(kSmMaskHr == offsetof(DeviceTables, mask_hr) - kFastOffset, "staged layout");

// Copies the staged part of the tables to the first 16 KiB boundary of the
// CTA's dynamic shared memory (all threads; the caller synchronises) and returns
// that address.  The launch must reserve kFastBytes + kSmAlign bytes for it.
__device__ __forceinline__ unsigned char* stage_fast_tables(const DeviceTables* tab, unsigned char* smem) {
    const uint32_t s = smem_u32(smem);
    unsigned char* base = smem + (((s + kSmAlign - 1) & ~(kSmAlign - 1)) - s);
    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(tab) + kFastOffset);
    uint4* dst = reinterpret_cast<uint4*>(base);
    for (uint32_t i = threadIdx.x; i < kFastBytes / 16; i += blockDim.x) dst[i] = src[i];
    return base;
}
constexpr uint32_t kTableSmemBytes = uint32_t(kFastBytes) + kSmAlign;

// PRMT pool of the p = 0 image, indexed by rank | c << 2:
//   c = 0: 0, 4, -4, 8     c = 1: 2, -2, 6, -6
constexpr uint32_t kPoolLo = 0x08FC0400u;
constexpr uint32_t kPoolHi = 0xFA06FE02u;
constexpr uint32_t kRank4Flags = 0x88888888u;

struct FastBlock {
    uint32_t y0[6];   // p = 0 image, int8 x 4, coordinate 4k+i in byte i of y0[k]
    uint32_t row1;    // rank rows of sections 1 and 3 (bit 3 of a nibble flags a rank-4 coordinate)
    uint32_t row3;
    uint32_t sel1;    // PRMT selectors (rank | c << 2 per nibble), for the fix-up
    uint32_t sel3;
    uint32_t p13;     // p << 13
    uint32_t goff;    // shared-memory address of the gain's half of the scale table (bit 7 = g)
};

// HI = false: w1 sits in bits 0..15 of `w1pair`; HI = true: in bits 16..31.
// sm_tab: shared-memory address of the staged tables, a multiple of 16 KiB, so
// that every index is merged with its table's address by the same LOP3 that
// masks it.
template <bool HI>
__device__ __forceinline__ void fast_decode(uint32_t sm_tab, uint32_t w0, uint32_t w1pair, FastBlock& out) {
    const uint32_t addr1 = ((w0 << 2) & 0x3FFCu) | (sm_tab + kSmRows);    // (i1 | r << 11) * 4
    const uint32_t addr3p = ((w0 >> 10) & 0x3FFCu) | (sm_tab + kSmRows);  // (i3 | q << 11) * 4
    const uint32_t a4 = ((w0 >> 22) & 0x3Cu) | (sm_tab + kSmMaskH);
    const uint32_t b4 = ((w0 >> 26) & 0x3Cu) | (sm_tab + kSmMaskH);
    uint32_t addr2, x4;
    if (HI) {
        addr2 = ((w1pair >> 14) & 0x1FFCu) | (sm_tab + kSmMid);
        x4 = ((w1pair >> 25) & 0x3Cu) | (sm_tab + kSmMaskHr);
        out.goff = ((w1pair >> 24) & 0x80u) | (sm_tab + kSmScale);
    } else {
        addr2 = ((w1pair << 2) & 0x1FFCu) | (sm_tab + kSmMid);
        x4 = ((w1pair >> 9) & 0x3Cu) | (sm_tab + kSmMaskHr);
        out.goff = ((w1pair >> 8) & 0x80u) | (sm_tab + kSmScale);
    }
    const uint32_t row1 = lds32(addr1);
    const uint32_t row2 = lds32(addr2);
    // delta = [i2 >= 1240]: bit 11 of i2 + 808, i.e. bit 13 of the byte offset; Eq. (3).
    // (the table bases are multiples of 8 KiB, so they do not disturb bits 0..12 of the sum)
    const uint32_t addr3 = addr3p ^ ((addr2 + 808u * 4u) & 0x2000u);
    const uint32_t row3 = lds32(addr3);
    const uint32_t ma = lds32(a4);
    const uint32_t mb = lds32(b4);
    const uint32_t mx = lds32(x4);
    const uint32_t sel1 = row1 ^ ma ^ mx;
    const uint32_t sel2 = row2 ^ mb ^ mx;
    const uint32_t sel3 = row3 ^ (ma ^ mb) ^ mx;
    out.y0[0] = prmt(kPoolLo, kPoolHi, sel1);
    out.y0[1] = prmt(kPoolLo, kPoolHi, sel1 >> 16);
    out.y0[2] = prmt(kPoolLo, kPoolHi, sel2);
    out.y0[3] = prmt(kPoolLo, kPoolHi, sel2 >> 16);
    out.y0[4] = prmt(kPoolLo, kPoolHi, sel3);
    out.y0[5] = prmt(kPoolLo, kPoolHi, sel3 >> 16);
    out.row1 = row1;
    out.row3 = row3;
    out.sel1 = sel1;
    out.sel3 = sel3;
    out.p13 = (addr1 ^ addr3p) & 0x2000u;  // r ^ q = p
}

// A flagged nibble (rank 4, stored as 8 | 2) makes PRMT return the sign fill of
// pool entry 2 (c = 0: -1) or 6 (c = 1: 0) instead of the rank-4 value
// (c = 0: -8, c = 1: 10).  Returns the coordinate inside the section, the
// amount to add to y0 there, and the change of sum(y0^2).
__device__ __forceinline__ void rank4_fix(uint32_t flags, uint32_t sel, int* j, int* dy, int* dsq) {
    const int bit = __ffs(int(flags)) - 1;  // 4 j + 3
    *j = bit >> 2;
    const bool c = (sel >> (bit - 1)) & 1u;
    *dy = c ? 10 : -7;    // 10 - 0, -8 - (-1)
    *dsq = c ? 100 : 63;  // 100 - 0, 64 - 1
}

}  // namespace tetra
