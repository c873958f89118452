// Host-side construction of the Tetra decode tables (Sec. 3.2-3.4) and of the
// derived lookup tables the sm_100a kernels stage in shared memory.
#pragma once
#include <cstddef>
#include <cstdint>

namespace tetra {

// The tables exactly as the paper lays them out (Sec. 3.4): 18,816 bytes.
struct PaperTables {
    uint32_t rows[4096];      // rank rows, class 0 then class 1, nibble j = rank of coordinate j
    uint8_t prefixes[128];    // [2*s8 + b1]
    uint16_t branches[1024];  // [16*s8 + b2] = middle byte | s16 << 8
    uint8_t suffixes[128];    // [2*s16 + b3]
    float rsqrt16m[32];       // 1/sqrt(16 m), entry 0 = 0
};
static_assert(sizeof(PaperTables) == 18816, "paper table blob is 18,816 bytes");

constexpr uint32_t kTableMagic = 0x54455442u;  // "TETB"
constexpr uint32_t kTableVersion = 7;
constexpr int kRank4Slots = 32;                // slots at the start of each class whose pool is patched
constexpr int kMiddleClass0 = 1240;            // N0 of Sec. 3.3 (checked at build)

// Everything tetra_build_table copies to the device, in one blob.
struct DeviceTables {
    PaperTables paper;          //     0: file-order decode (tetra_decode_blocks, paper-design GEMV)
    float gain[2];              // 18816
    uint32_t magic;             // 18824
    uint32_t version;           // 18828
    // ---- fast path: everything below is staged in shared memory ------------
    // Rank rows for PRMT lookup, class by class in the permuted order of
    // row_perm: nibble j = rank << 1 (ranks 0..3; bit 0 is where the pattern bit
    // goes).  The first 32 slots of each class hold the rows with a coordinate of
    // rank 4 (stored there as rank 2) and, as fillers, rows that use ranks 0 and
    // 1 only: for those slots the kernels swap in a PRMT pool word whose rank-2
    // entries are the rank-4 values.
    // (the kernels place this part on a 16 KiB boundary of shared memory, so each
    //  sub-table's offset can be OR-ed into an index instead of added)
    uint32_t rows_fast[4096];   // +0
    uint32_t mid_fast[2048];    // +16384: rows_fast[mix(i2)], indexed by i2 directly
    float scale[2][32][4];      // +24576: -gain[g] / sqrt(16 m) in entry [0][m][2 g] (the second half is spare):
                                //         16 bytes per m, so that the block's squared norm 16 m is the byte
                                //         offset itself, and the two gains 8 bytes apart, so that lanes with
                                //         nearby m or different g read different banks.  Minus: the fast
                                //         decoder emits -y.
    // Pattern-byte masks of the Turyn coordinates: bit 4j set where the
    // Hamming word has coordinate j set; H for a and b, H' for x.
    uint32_t mask_h[16];        // +25600
    uint32_t mask_hr[16];       // +25664
    uint32_t pad_[16];          // +25728 (spare)
    // ---- pack-time only (global memory) ------------------------------------
    // 12 trellis bits (s8 | b1<<6 | b2<<7 | b3<<11) -> Turyn coordinates a | b<<4 | x<<8.
    uint16_t trellis_to_abx[4096];
    // row_perm[cls][i]: slot of file-order row 2048 cls + i inside its class of rows_fast.
    uint16_t row_perm[2][2048];
};

constexpr size_t kFastOffset = offsetof(DeviceTables, rows_fast);
constexpr size_t kFastBytes = offsetof(DeviceTables, trellis_to_abx) - kFastOffset;
static_assert(kFastOffset % 16 == 0 && kFastBytes % 16 == 0, "staged part must be 16-byte copyable");

// Fills `out` (gain from gain2, or the defaults when null).  Returns 0, or a
// negative number naming the structural check that failed (never expected).
int build_device_tables(DeviceTables* out, const float* gain2);

}  // namespace tetra
