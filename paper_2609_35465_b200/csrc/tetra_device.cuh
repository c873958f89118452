// Device-side decoders for Tetra words (sm_100a).
//
// Two decoders live here:
//   * decode_file_word: the six-load decode of Sec. 3.4 (Fig. "decode") on a
//     word in file order, reading the paper-format tables.  Used by
//     tetra_decode_blocks and by the paper-design GEMV.
//   * the fast decoder: works on the re-ordered 48-bit device word written by
//     tetra_pack_codes and on tables staged in shared memory.  It produces the
//     lattice point (negated) as packed int8, four coordinates per register and
//     one PRMT per four: a selector nibble is c | rank << 1 and the 8-byte PRMT
//     pool holds the rank lists of Sec. 3.3 for the block's parity p.
//     Branch-free: rows with a coordinate of rank 4 sit in the first 32 slots of
//     their class, and for those slots one select swaps in a pool word whose
//     rank-2 entries are the rank-4 values.
#pragma once
#include <cstdint>
#include <cuda_fp16.h>
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
// Programmatic dependent launch.  Every GEMV kernel lets the next kernel of the
// stream start early (pdl_release) and waits for its own predecessor only when
// it first touches data a predecessor may have produced (pdl_wait): tables and
// codes are constants of the model, activations are not.  Both are no-ops for a
// kernel launched without the attribute.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

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
//   w0: [0..10] i1'  [11] r  [12..22] i3'  [23] q = p^r  [24..27] a  [28..31] b
//   w1: [0..10] i2  [11..14] x  [15] g
// i1', i3' are the row indices after the per-class permutation row_perm (class r
// for section 1, class r3 = p^r^delta for section 3).  (a, b, x) are the Turyn
// coordinates of the trellis path: the three pattern bytes are h(a)+h'(x),
// h(b)+h'(x), h(a)+h(b)+h'(x).
// ---------------------------------------------------------------------------
__device__ __forceinline__ void file_to_device_word(uint64_t w, const DeviceTables* tab, uint32_t* w0, uint32_t* w1) {
    uint32_t i1 = uint32_t(w & 0x7FF), i3 = uint32_t((w >> 22) & 0x7FF);
    const uint32_t i2 = uint32_t((w >> 11) & 0x7FF);
    const uint32_t path = uint32_t((w >> 33) & 0xFFF);
    const uint32_t p = uint32_t((w >> 45) & 1), r = uint32_t((w >> 46) & 1), g = uint32_t((w >> 47) & 1);
    const uint32_t r3 = p ^ r ^ uint32_t(i2 >= uint32_t(kMiddleClass0));  // Eq. (3)
    i1 = tab->row_perm[r][i1];
    i3 = tab->row_perm[r3][i3];
    const uint32_t abx = tab->trellis_to_abx[path];
    *w0 = i1 | (r << 11) | (i3 << 12) | ((p ^ r) << 23) | ((abx & 0xFFu) << 24);
    *w1 = i2 | ((abx >> 8) << 11) | (g << 15);
}

// Byte offsets of the staged tables inside the shared-memory copy of the fast part.
constexpr uint32_t kSmRows = 0;
constexpr uint32_t kSmMid = 16384;
constexpr uint32_t kSmScale = 24576;
constexpr uint32_t kSmMaskH = 25600;
constexpr uint32_t kSmMaskHr = 25664;
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
// The same copy with cp.async (16 bytes per request, all of a thread's requests in flight at once);
// the caller commits and waits for the group and synchronises the CTA before the tables are read.
__device__ __forceinline__ unsigned char* stage_fast_tables_async(const DeviceTables* tab, unsigned char* smem) {
    const uint32_t s = smem_u32(smem);
    const uint32_t pad = ((s + kSmAlign - 1) & ~(kSmAlign - 1)) - s;
    const char* src = reinterpret_cast<const char*>(tab) + kFastOffset;
    for (uint32_t i = threadIdx.x; i < kFastBytes / 16; i += blockDim.x)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(s + pad + 16u * i), "l"(src + 16u * i));
    return smem + pad;
}
constexpr uint32_t kTableSmemBytes = uint32_t(kFastBytes) + kSmAlign;

// PRMT pools.  A selector nibble is c | rank << 1 (c: the coordinate's pattern bit, ranks 0..3 of the
// lists of Sec. 3.3), so the low pool word serves ranks 0 and 1 and the high word ranks 2 and 3:
//   lo = { r0c0, r0c1, r1c0, r1c1 }    hi = { r2c0, r2c1, r3c0, r3c1 }
// The pools hold MINUS the coordinate (the scale table holds minus the block scale, so products come
// out with the right sign):
//   p = 0:  y = 0, 2 | 4, -2 | -4, 6 | 8, -6        p = 1:  y = 1, -1 | -3, 3 | 5, -5 | -7, 7
// A row with a coordinate of rank 4 (y = -8, 10 for p = 0; 9, -9 for p = 1) stores it as rank 2 and
// sits in the first kRank4Slots slots of its class; for those slots the two rank-2 bytes of the high
// word become the rank-4 values, which in this sign convention is the same XOR for both parities.
constexpr uint32_t kPool0Lo = 0x02FCFE00u, kPool0Hi = 0x06F8FA04u;
constexpr uint32_t kPool1Lo = 0xFD0301FFu, kPool1Hi = 0xF90705FBu;
constexpr uint32_t kRank4Patch = 0x00000C0Cu;
constexpr uint32_t kSpecialAddrMask = uint32_t(2048 - kRank4Slots) * 4u;  // zero <=> slot < kRank4Slots
static_assert(kRank4Slots == 32 && kSpecialAddrMask == 0x1F80u, "special slots are the first 32 of a class");

struct FastBlock {
    uint32_t y[6];  // MINUS the lattice point, int8 x 4, coordinate 4k+i in byte i of y[k]
    uint32_t goff;  // shared-memory address of the scale table plus 8 g (the gain's column of the table)
};

// HI = false: w1 sits in bits 0..15 of `w1pair`; HI = true: in bits 16..31.
// sm_tab: shared-memory address of the staged tables, a multiple of 16 KiB, so
// that every index is merged with its table's address by the same LOP3 that
// masks it.
template <bool HI>
__device__ __forceinline__ void fast_decode(uint32_t sm_tab, uint32_t w0, uint32_t w1pair, FastBlock& out) {
    const uint32_t addr1 = ((w0 << 2) & 0x3FFCu) | (sm_tab + kSmRows);    // (i1' | r << 11) * 4
    const uint32_t addr3p = ((w0 >> 10) & 0x3FFCu) | (sm_tab + kSmRows);  // (i3' | q << 11) * 4
    const uint32_t a4 = ((w0 >> 22) & 0x3Cu) | (sm_tab + kSmMaskH);
    const uint32_t b4 = ((w0 >> 26) & 0x3Cu) | (sm_tab + kSmMaskH);
    uint32_t addr2, x4;
    if (HI) {
        addr2 = ((w1pair >> 14) & 0x1FFCu) | (sm_tab + kSmMid);
        x4 = ((w1pair >> 25) & 0x3Cu) | (sm_tab + kSmMaskHr);
        out.goff = ((w1pair >> 28) & 8u) | (sm_tab + kSmScale);
    } else {
        addr2 = ((w1pair << 2) & 0x1FFCu) | (sm_tab + kSmMid);
        x4 = ((w1pair >> 9) & 0x3Cu) | (sm_tab + kSmMaskHr);
        out.goff = ((w1pair >> 12) & 8u) | (sm_tab + kSmScale);
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
    // p = r ^ q sits at bit 13 of both row addresses: one test, two selects for the pools
    const bool p = ((addr1 ^ addr3p) & 0x2000u) != 0;
    const uint32_t lo = p ? kPool1Lo : kPool0Lo;
    const uint32_t hi = p ? kPool1Hi : kPool0Hi;
    const uint32_t hix = hi ^ kRank4Patch;
    const uint32_t hi1 = (addr1 & kSpecialAddrMask) ? hi : hix;
    const uint32_t hi3 = (addr3p & kSpecialAddrMask) ? hi : hix;
    out.y[0] = prmt(lo, hi1, sel1);
    out.y[1] = prmt(lo, hi1, sel1 >> 16);
    out.y[2] = prmt(lo, hi, sel2);
    out.y[3] = prmt(lo, hi, sel2 >> 16);
    out.y[4] = prmt(lo, hi3, sel3);
    out.y[5] = prmt(lo, hi3, sel3 >> 16);
}

// ---------------------------------------------------------------------------
// Activations
// ---------------------------------------------------------------------------
// Fixed-point image of one block column of activations (20 words).
// step = 2^(E-22) with 2^E <= max|x| < 2^(E+1); q_j = rint(x_j / step), |q_j| < 2^23,
// stored as three byte planes (bits 23..16 signed, 15..8 and 7..0 unsigned), four
// coordinates per 32-bit word: words 0..5 high, 6..11 middle, 12..17 low plane;
// word 18 = step (float), word 19 = sum(q_j).  A float16 x_j is held exactly when
// |x_j| >= 2^(E-12); smaller ones are rounded to a multiple of the step.  If a value
// is NaN or infinite the step is NaN (and the planes zero).
__device__ __forceinline__ void quantise_column(const __half* __restrict__ x, int K, int c, uint32_t out[20]) {
    float v[24];
    const int k0 = 24 * c;
    if (k0 + 24 <= K && ((reinterpret_cast<uintptr_t>(x) & 15) == 0)) {  // 48-byte column, 16-byte aligned
        const uint4* src = reinterpret_cast<const uint4*>(x + k0);
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint4 u = __ldg(src + i);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const __half2 h = *reinterpret_cast<const __half2*>(&w[j]);
                v[8 * i + 2 * j] = __low2float(h);
                v[8 * i + 2 * j + 1] = __high2float(h);
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < 24; ++j) v[j] = k0 + j < K ? __half2float(x[k0 + j]) : 0.f;
    }
    // largest magnitude, compared as bit patterns (same order as the values for non-negative floats):
    // a NaN or an infinity, whose exponent field is all ones, then counts as the largest
    uint32_t mxb = 0u;
#pragma unroll
    for (int j = 0; j < 24; ++j) mxb = max(mxb, __float_as_uint(v[j]) & 0x7FFFFFFFu);
    const bool finite = mxb < 0x7F800000u;
    const uint32_t e = mxb >> 23;  // biased exponent of the largest
    // A NaN or an infinity among the 24 values makes the step NaN, so every product with this column, and
    // with it every output row that reads the column, comes out NaN instead of a finite, wrong number.
    const float step = !finite ? __uint_as_float(0x7FC00000u) : (mxb ? __uint_as_float((e - 22u) << 23) : 0.f);
    const float inv = (finite && mxb) ? __uint_as_float((276u - e) << 23) : 0.f;
    int sum = 0;
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        uint32_t hi = 0, mid = 0, lo = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int q = __float2int_rn(v[4 * k + i] * inv);
            sum += q;
            hi |= (uint32_t(q >> 16) & 0xFFu) << (8 * i);
            mid |= (uint32_t(q >> 8) & 0xFFu) << (8 * i);
            lo |= (uint32_t(q) & 0xFFu) << (8 * i);
        }
        out[k] = hi;
        out[6 + k] = mid;
        out[12 + k] = lo;
    }
    out[18] = __float_as_uint(step);
    out[19] = uint32_t(sum);
}


}  // namespace tetra
