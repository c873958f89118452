// Decode-and-multiply for 2..16 activation vectors at once (Eq. (2), Sec. 5.1): k_gemv_batched (5..16
// vectors, described first) and k_gemv_few (2..4 vectors, further down).
//
// A block is decoded once and multiplied with every vector, so the decode cost
// is shared.  The products over a block's 24 coordinates for up to 16 vectors
// are a small dense contraction, int8 x int8 -> int32, and run on the tensor
// cores (mma.sync m16n8k32); everything around it (field extraction, table
// lookups, per-block scale, FP32 accumulation) is the batch-1 decoder.
//
// Thread layout: a warp owns two row blocks of 16 rows, a CTA of 16 warps a tile group of 512 rows, and a
// warp walks the block columns four at a time; such a (tile group, four columns) cell is the unit of work,
// and the CTAs take equal contiguous ranges of the tile-group-major cell order.  The codes of a warp's pass
// (four row groups x three parts x four columns) arrive through the warp's own cp.async ring, one pass
// ahead.  In one pass lane l decodes four blocks (row l % 16 of row block j % 2, column l / 16 + 2 (j / 2),
// j = 0..3) and writes each block's 24 int8 coordinates and its scale as a row of a shared-memory tile;
// the warp then loads the tiles as MMA A fragments with ldmatrix and multiplies them with the three int8
// planes of the activations' 24-bit fixed-point image (B fragments, read once per column and used for both
// row blocks; coordinates 24..31 of the image are zero, so the tile's bytes there do not matter).  The image
// of the CTA's next 32 (column, vector group) pairs is built by the CTA itself, in shared memory: once for
// most calls (behind the first pass's decode), again behind two CTA barriers when the CTA's range is
// longer; between those the warps never wait for one another.  The int32 results of the planes are
// combined exactly, converted once, scaled by block scale x activation step and added into FP32
// accumulators that the lane keeps for its (row, vector) pairs: no cross-lane reduction is needed.  When a
// CTA's range leaves a tile group, its partial sums go to the scratch area as one piece; a second, small
// kernel adds the pieces of every tile group in CTA order (fixed order, no atomics, no flags), applies the
// row scale and the tail.  The only waits are CTA barriers, cp.async groups and griddepcontrol.wait.
#include <cuda_fp16.h>

#include "tetra_gemv_common.cuh"

namespace tetra {

constexpr int kBatThreads = 512;
constexpr int kBatWarps = kBatThreads / 32;
#ifndef TETRA_BAT_RB1
#define TETRA_BAT_RB1 2  // row blocks per warp, batch <= 8
#endif
#ifndef TETRA_BAT_RB2
#define TETRA_BAT_RB2 2  // row blocks per warp, batch 9..16
#endif
constexpr int kPassTiles = 8;  // 16-row x 1-column tiles per warp and pass (four blocks per lane)
// Activation image per block column and vector group n (vectors 8 n .. 8 n + 7): two 16-byte chunks per
// lane, stored chunk-major ([chunk][lane][4 words]) so that a 128-bit access per chunk is contiguous over
// the warp:
//   chunk 2 n     = B-fragment registers (plane 0, h 0), (0, 1), (1, 0), (1, 1)
//   chunk 2 n + 1 = (2, 0), (2, 1), step of vector 8 n + 2 t, step of vector 8 n + 2 t + 1
// where the lane multiplies with vector 8 n + lane / 4, t = lane % 4, register h = 0 holds coordinates
// 4 t .. 4 t + 3 and h = 1 coordinates 16 + 4 t .. 16 + 4 t + 3 (24..31 and unused vectors are zero), and
// the steps are those of the lane's two result columns.  A column takes ng x 1 KiB (ng = 1 or 2 groups).
// The image lives in shared memory only: the CTA builds it for a chunk of its passes at a time.
constexpr int kBatGroupWords = 2 * 32 * 4;

// One thread per (block column of a pass, vector, t) builds the words of lane (vector % 8) * 4 + t: the
// thread reads the (up to) eight activations that lane multiplies with, the column's largest magnitude is
// found over the four threads of the vector (two shuffles), and the 24-bit fixed-point values are split
// into the three int8 planes.  A float16 x_j is held exactly when |x_j| >= 2^(E-12), E the exponent of the
// column's largest magnitude; smaller ones are rounded to a multiple of the step 2^(E-22).
struct ImageTask {
    float v[8];  // coordinates 4 t .. 4 t + 3 and (t < 2) 16 + 4 t .. 19 + 4 t of the column
};
__device__ __forceinline__ void image_load(const __half* __restrict__ x, int K, int batch, int col, int vec, int t,
                                           ImageTask& T) {
    const __half* xv = x + size_t(vec) * K;
    const int k0 = 24 * col + 4 * t;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        T.v[i] = (vec < batch && k0 + i < K) ? __half2float(__ldg(xv + k0 + i)) : 0.f;
        T.v[4 + i] = (vec < batch && t < 2 && k0 + 16 + i < K) ? __half2float(__ldg(xv + k0 + 16 + i)) : 0.f;
    }
}
// group_base: shared-memory address of the column's 1 KiB group for the vector's group of eight.
__device__ __forceinline__ void image_store(const ImageTask& T, uint32_t group_base, int vec, int t) {
    // largest magnitude as a bit pattern (a NaN or an infinity then counts as the largest)
    uint32_t mxb = 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) mxb = max(mxb, __float_as_uint(T.v[i]) & 0x7FFFFFFFu);
    mxb = max(mxb, __shfl_xor_sync(0xFFFFFFFFu, mxb, 1));
    mxb = max(mxb, __shfl_xor_sync(0xFFFFFFFFu, mxb, 2));
    const bool finite = mxb < 0x7F800000u;
    const uint32_t e = mxb >> 23;  // biased exponent of the largest
    // a NaN or an infinity in the column makes its step NaN: every row that reads the column comes out NaN
    const float step = !finite ? __uint_as_float(0x7FC00000u) : (mxb ? __uint_as_float((e - 22u) << 23) : 0.f);
    const float inv = (finite && mxb) ? __uint_as_float((276u - e) << 23) : 0.f;
    uint32_t b[3][2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint32_t hi = 0, mid = 0, lo = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int q = __float2int_rn(T.v[4 * h + i] * inv);
            hi |= (uint32_t(q >> 16) & 0xFFu) << (8 * i);
            mid |= (uint32_t(q >> 8) & 0xFFu) << (8 * i);
            lo |= (uint32_t(q) & 0xFFu) << (8 * i);
        }
        b[0][h] = hi;
        b[1][h] = mid;
        b[2][h] = lo;
    }
    const int g = vec & 7, ln = g * 4 + t;
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(group_base + ln * 16), "r"(b[0][0]), "r"(b[0][1]),
                 "r"(b[1][0]), "r"(b[1][1]) : "memory");
    asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(group_base + 512 + ln * 16), "r"(b[2][0]), "r"(b[2][1]) : "memory");
    // the step goes to the eight lanes whose results belong to this vector: lane % 4 = (vec % 8) / 2, any lane / 4
#pragma unroll
    for (int gg = 2 * t; gg < 2 * t + 2; ++gg)
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(group_base + 512 + (gg * 4 + (g >> 1)) * 16 + 8 + 4 * (vec & 1)), "f"(step)
                     : "memory");
}

__device__ __forceinline__ void mma_s8s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(0));
}
__device__ __forceinline__ void mma_s8u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(0));
}

constexpr int kTileRow = 48;                // bytes per tile row: 24 coordinates, scale, 20 pad
constexpr int kTileBytes = 16 * kTileRow;   // (48-byte rows keep ldmatrix and the tile stores conflict-free)
constexpr int kBatWarpTiles = kPassTiles * kTileBytes;  // coordinate tiles (a row: 24 coordinates, the block scale, pad)
constexpr int kBatColBytesPerGroup = kBatGroupWords * 4;                   // image of one column, per ng
// Code ring of a warp: two slots of one pass (the warp's four row groups x three parts x four columns x 16
// bytes); a row group takes 224 bytes, so that the loads of a pass (two row groups x two parts x two
// columns x four words per instruction) fall into different banks.
constexpr uint32_t kBatRingGroup = 224, kBatRingSlot = 4 * kBatRingGroup;
constexpr int kBatWarpSmem = kBatWarpTiles + 2 * int(kBatRingSlot);
constexpr int kImageGroups = 32;  // (column, vector group) pairs of the activation image held at a time: 32 KiB

__device__ __forceinline__ void lds128(uint32_t saddr, uint32_t (&v)[4]) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(saddr));
}

// CTA that owns cell x when CTA i owns cells [i * cells / ctas, (i + 1) * cells / ctas).
__device__ __forceinline__ uint32_t cta_of_cell(uint32_t x, uint32_t ctas, uint32_t cells) {
    return uint32_t(((uint64_t(x) + 1) * ctas - 1) / cells);
}

// NG: vector groups of eight, 1 (batch <= 8) or 2.  A warp owns two 16-row blocks (RB = 2), the CTA's 16
// warps a tile group of 512 rows; a cell is a tile group x four block columns, one pass of every warp.
// The CTAs take equal contiguous ranges of the tile-group-major cell order.  Between the image barriers the
// warps run on their own: codes arrive through the warp's cp.async ring one pass ahead.
template <int NG, int RB>
__global__ void __launch_bounds__(kBatThreads, 1)
k_gemv_batched(const DeviceTables* __restrict__ tab, const unsigned char* __restrict__ codes,
               const __half* __restrict__ x, int N, int K, int B, int batch, float* __restrict__ partials, int tile_groups, int col_groups) {
    static_assert(RB == 2, "the ring and the lane mapping are laid out for two row blocks per warp");
    constexpr int PC = kPassTiles / RB;          // block columns per pass
    constexpr int CP = kImageGroups / (PC * NG); // passes per image chunk
    constexpr int kPieceFloats = RB * 128 * NG;  // partial results of one warp: 16 RB rows x 8 NG vectors
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pdl_release();
    // the tables start towards shared memory first; they are waited for together with the first pass's codes
    unsigned char* smem = stage_fast_tables_async(tab, smem_raw);
    const uint32_t sm_tab = smem_u32(smem);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // per warp: eight 16-row tiles of coordinates and block scales (tile rb * PC + column), the code ring;
    // after the warps' areas, the activation image of a chunk of passes
    unsigned char* tiles = smem + kFastBytes + warp * kBatWarpSmem;
    const uint32_t ring = smem_u32(tiles) + uint32_t(kBatWarpTiles);
    const uint32_t image = smem_u32(smem + kFastBytes + kBatWarps * kBatWarpSmem);
    const int row16 = lane & 15, colsel = lane >> 4;

    const int row_groups = (N + 7) / 8;
    const uint32_t Bu = uint32_t(B);
    const int g = lane >> 2, t4 = lane & 3;  // MMA fragment coordinates
    const uint32_t tile_addr = smem_u32(tiles);
    // ldmatrix: lane provides the address of row (lane % 8) of 8x8 matrix (lane / 8):
    // matrices = (rows 0-7, bytes 0-15), (rows 8-15, bytes 0-15), (rows 0-7, bytes 16-31), (rows 8-15, bytes 16-31)
    const uint32_t ldm_off = uint32_t((((lane >> 3) & 1) * 8 + (lane & 7)) * kTileRow + (lane >> 4) * 16);
    // block j of the lane in a pass: row row16 of row block j % 2, column colsel + 2 (j / 2); its words in a slot
    const uint32_t lane_w0 = uint32_t(row16 >> 3) * kBatRingGroup + uint32_t((row16 >> 2) & 1) * 64u + uint32_t(colsel) * 16u +
                             uint32_t(row16 & 3) * 4u;
    const uint32_t lane_w1 = uint32_t(row16 >> 3) * kBatRingGroup + 128u + uint32_t(colsel) * 16u + uint32_t(row16 & 7) * 2u;
    // the lane's copies of a pass: 48 pieces of 16 bytes, (row group, part) = piece / 4, column = piece % 4
    const uint32_t cp0_gp = uint32_t(lane >> 2), cp1_gp = 8u + uint32_t(lane >> 2), cp_col = uint32_t(lane & 3);
    const uint32_t cp0_dst = (cp0_gp / 3u) * kBatRingGroup + (cp0_gp % 3u) * 64u + cp_col * 16u;
    const uint32_t cp1_dst = (cp1_gp / 3u) * kBatRingGroup + (cp1_gp % 3u) * 64u + cp_col * 16u;

    const uint32_t ctas = gridDim.x, cells = uint32_t(tile_groups) * uint32_t(col_groups), CG = uint32_t(col_groups);
    const uint32_t cell_begin = uint32_t(uint64_t(blockIdx.x) * cells / ctas);
    const uint32_t cell_end = uint32_t((uint64_t(blockIdx.x) + 1) * cells / ctas);
    uint32_t tg = cell_begin / CG, cg = cell_begin - tg * CG;

    // the codes of the warp's pass in cell (ftg, fcg) into ring slot `slot`; what lies outside the matrix is zero
    auto fetch = [&](uint32_t ftg, uint32_t fcg, uint32_t slot) {
        const uint32_t G0 = (ftg * kBatWarps + uint32_t(warp)) * (2 * RB);  // first of the warp's four row groups
        const uint32_t col = fcg * PC + cp_col;
        const bool in = col < Bu;
        const uint4* base = reinterpret_cast<const uint4*>(codes) + size_t(G0) * 3 * Bu + (in ? col : 0u);
        const uint32_t dst = ring + slot * kBatRingSlot;
        const bool have0 = in && G0 + cp0_gp / 3u < uint32_t(row_groups);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst + cp0_dst),
                     "l"(have0 ? base + size_t(cp0_gp) * Bu : reinterpret_cast<const uint4*>(codes)), "r"(have0 ? 16u : 0u));
        if (lane < 16) {
            const bool have1 = in && G0 + cp1_gp / 3u < uint32_t(row_groups);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst + cp1_dst),
                         "l"(have1 ? base + size_t(cp1_gp) * Bu : reinterpret_cast<const uint4*>(codes)), "r"(have1 ? 16u : 0u));
        }
        asm volatile("cp.async.commit_group;");
    };
    if (cell_begin < cell_end) fetch(tg, cg, 0);
    else asm volatile("cp.async.commit_group;");
    pdl_wait();  // x may come from the preceding kernel; the partial results of an earlier call have been read

    // Image tasks of a chunk of CP passes: task (pass i of the chunk, column cs, vector group n) = a warp's worth
    // of threads; the 16 warps take two tasks each.
    auto image_task_load = [&](uint32_t first_cell, int id, ImageTask& T) {
        const uint32_t cell = first_cell + uint32_t(id / (PC * NG));
        if (cell < cell_end) image_load(x, K, batch, int(cell % CG) * PC + (id / NG) % PC, 8 * (id % NG) + (lane >> 2), lane & 3, T);
    };
    auto image_task_store = [&](uint32_t first_cell, int id, const ImageTask& T) {
        const uint32_t cell = first_cell + uint32_t(id / (PC * NG));
        if (cell < cell_end) image_store(T, image + uint32_t(id) * 1024u, 8 * (id % NG) + (lane >> 2), lane & 3);
    };
    ImageTask task0, task1;
    image_task_load(cell_begin, warp, task0);
    image_task_load(cell_begin, warp + kBatWarps, task1);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();  // tables staged, tile padding written

    float acc[RB][NG][4];
#pragma unroll
    for (int rb = 0; rb < RB; ++rb)
#pragma unroll
        for (int n = 0; n < NG; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[rb][n][i] = 0.f;

    for (uint32_t cell = cell_begin; cell < cell_end; ++cell) {
        const uint32_t pass = cell - cell_begin, slot = pass & 1u, in_chunk = pass % CP;
        const bool active = (int(tg) * kBatWarps + warp) * (16 * RB) < N;  // warp-uniform
        uint32_t ntg = tg, ncg = cg + 1;
        if (ncg == CG) { ncg = 0; ++ntg; }
        if (in_chunk == 0 && pass > 0) {  // CTA-uniform: the image of the next chunk of passes replaces the old one
            __syncthreads();
            image_task_load(cell, warp, task0);
            image_task_load(cell, warp + kBatWarps, task1);
            image_task_store(cell, warp, task0);
            image_task_store(cell, warp + kBatWarps, task1);
            __syncthreads();
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();  // every lane's copies have landed, and every lane has left the other slot
        if (cell + 1 < cell_end) fetch(ntg, ncg, slot ^ 1u);
        if (active) {
            const uint32_t src = ring + slot * kBatRingSlot;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t w0, w1;
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w0) : "r"(src + lane_w0 + (j % RB) * 2 * kBatRingGroup + (j / RB) * 32));
                asm volatile("ld.shared.u16 %0, [%1];" : "=r"(w1) : "r"(src + lane_w1 + (j % RB) * 2 * kBatRingGroup + (j / RB) * 32));
                FastBlock fb;
                fast_decode<false>(sm_tab, w0, w1, fb);
                int n2 = int(fb.goff);  // the squared norm on top of the gain's column of the scale table: the scale's address
#pragma unroll
                for (int k = 0; k < 6; ++k) n2 = dp4a_ss(fb.y[k], fb.y[k], n2);
                const float scale = lds32f(uint32_t(n2));  // -gain[g] / sqrt(16 m), with -y in the tile
                const int tile_id = (j % RB) * PC + 2 * (j / RB);  // + colsel
                unsigned char* dst = tiles + (tile_id + colsel) * kTileBytes + row16 * kTileRow;
                // coordinates 24..31 of a tile row meet zeros in the activation image, so those eight bytes
                // need not be zero: the block's scale rides there
                *reinterpret_cast<uint4*>(dst) = make_uint4(fb.y[0], fb.y[1], fb.y[2], fb.y[3]);
                *reinterpret_cast<uint4*>(dst + 16) = make_uint4(fb.y[4], fb.y[5], __float_as_uint(scale), 0u);
            }
        }
        if (pass == 0) {  // the first chunk's image: its loads were issued before the first pass was decoded
            image_task_store(cell_begin, warp, task0);
            image_task_store(cell_begin, warp + kBatWarps, task1);
            __syncthreads();
        }
        if (active) {
            __syncwarp();
            const uint32_t img = image + in_chunk * (PC * NG * 1024u) + lane * 16;
#pragma unroll
            for (int cs = 0; cs < PC; ++cs) {
                uint32_t q0[NG][4], q1[NG][4];
#pragma unroll
                for (int n = 0; n < NG; ++n) {
                    lds128(img + (cs * NG + n) * 1024, q0[n]);
                    lds128(img + (cs * NG + n) * 1024 + 512, q1[n]);
                }
#pragma unroll
                for (int rb = 0; rb < RB; ++rb) {
                    const int tile_id = rb * PC + cs;
                    uint32_t a[4];
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                                 : "r"(tile_addr + tile_id * kTileBytes + ldm_off));
                    const float s_lo = *reinterpret_cast<const float*>(tiles + tile_id * kTileBytes + g * kTileRow + 24);
                    const float s_hi = *reinterpret_cast<const float*>(tiles + tile_id * kTileBytes + (g + 8) * kTileRow + 24);
#pragma unroll
                    for (int n = 0; n < NG; ++n) {
                        int dh[4], dm[4], dl[4];
                        mma_s8s8(dh, a, q0[n][0], q0[n][1]);
                        mma_s8u8(dm, a, q0[n][2], q0[n][3]);
                        mma_s8u8(dl, a, q1[n][0], q1[n][1]);
                        const float step_even = __uint_as_float(q1[n][2]), step_odd = __uint_as_float(q1[n][3]);
                        // this lane's results: rows g (i = 0, 1) and g + 8 (i = 2, 3), vectors 8 n + 2 t4 + (i & 1)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            int dot;  // dh * 65536 + dm * 256 + dl, exact (|dot| < 2^31), on the multiply-add pipe
                            asm("mad.lo.s32 %0, %1, 256, %2;" : "=r"(dot) : "r"(dm[i]), "r"(dl[i]));
                            asm("mad.lo.s32 %0, %1, 65536, %0;" : "+r"(dot) : "r"(dh[i]));
                            acc[rb][n][i] = fmaf(float(dot), (i < 2 ? s_lo : s_hi) * ((i & 1) ? step_odd : step_even),
                                                 acc[rb][n][i]);
                        }
                    }
                }
            }
            __syncwarp();  // the fragments have been read before the next pass overwrites the tiles
        }
        if (cell + 1 == cell_end || ntg != tg) {  // CTA-uniform: this CTA's piece of tile group tg is complete
            // pieces are numbered blockIdx.x + tg: unique, and increasing along the cell order
            float* mine = partials + (size_t(blockIdx.x + tg) * kBatWarps + warp) * kPieceFloats;
#pragma unroll
            for (int rb = 0; rb < RB; ++rb)
#pragma unroll
                for (int n = 0; n < NG; ++n)
#pragma unroll
                    for (int i = 0; i < 4; i += 2) {
                        *reinterpret_cast<float2*>(mine + (16 * rb + g + (i < 2 ? 0 : 8)) * (8 * NG) + 8 * n + 2 * t4) =
                            make_float2(acc[rb][n][i], acc[rb][n][i + 1]);
                        acc[rb][n][i] = 0.f;
                        acc[rb][n][i + 1] = 0.f;
                    }
        }
        tg = ntg;
        cg = ncg;
    }
}

// ---------------------------------------------------------------------------------------------
// Two to four vectors: the same cells, rings, image chunks and pieces as k_gemv_batched, but no shared-memory
// tile between decoder and tensor cores.  Lane 4 q + t decodes, for each of the warp's two row blocks, rows
// 2 q and 2 q + 1 at column t of the pass's four columns; the MMA takes eight coordinates of both blocks
// from every lane as A (rows q and q + 8), and B is block diagonal -- column 2 t + plane of B is zero outside
// the k range that lane t feeds -- so D[q][2 t + plane] is the dot product of lane (q, t)'s own block with
// its own column's activation plane and arrives in that same lane.  Three MMAs (coordinate pairs) times two
// B sets (unsigned middle and low planes; signed high plane) per vector and row block.  The activation
// image holds, per (column quad, vector), the B fragments as they are read: three 128-byte lines (one per
// coordinate pair: bytes 0..63 middle and low planes, entry 2 t + plane; 64..95 high plane, entry t;
// 96..103 zero, read by the lanes whose part of B is zero), the four columns' steps at 104 + 4 t of line 0.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kQuadBytes = 384;
constexpr int kFewMaxVectors = 4;
constexpr int kFewChunkPasses = 16;  // passes whose image is held at a time: 16 x 4 vectors x 384 bytes = 24 KiB

__device__ __forceinline__ void mma_bd(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1, const int (&c)[4], bool b_signed) {
    if (b_signed)
        asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
            : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]));
    else
        asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
            : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]));
}

template <int V>
__global__ void __launch_bounds__(kBatThreads, 1)
k_gemv_few(const DeviceTables* __restrict__ tab, const unsigned char* __restrict__ codes, const __half* __restrict__ x,
           int N, int K, int B, float* __restrict__ partials, int tile_groups, int col_groups) {
    constexpr int RB = 2, PC = 4, CP = kFewChunkPasses;
    constexpr int kPieceFloats = RB * 128;  // the piece layout of k_gemv_batched<1, 2>: 32 rows x 8 vector slots
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pdl_release();
    unsigned char* smem = stage_fast_tables_async(tab, smem_raw);
    const uint32_t sm_tab = smem_u32(smem);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = lane >> 2, t = lane & 3;
    const uint32_t ring = smem_u32(smem + kFastBytes) + uint32_t(warp) * (2 * kBatRingSlot);
    const uint32_t image = smem_u32(smem + kFastBytes) + uint32_t(kBatWarps) * (2 * kBatRingSlot);
    unsigned char* image_ptr = smem + kFastBytes + kBatWarps * (2 * kBatRingSlot);
    const int row_groups = (N + 7) / 8;
    const uint32_t Bu = uint32_t(B);
    // the lane's words in a slot: rows 2 q, 2 q + 1 of row block rb sit in row group 2 rb + q / 4, part (q / 2) % 2
    const uint32_t lane_w0 = uint32_t(q >> 2) * kBatRingGroup + uint32_t((q >> 1) & 1) * 64u + uint32_t(t) * 16u + uint32_t(q & 1) * 8u;
    const uint32_t lane_w1 = uint32_t(q >> 2) * kBatRingGroup + 128u + uint32_t(t) * 16u + uint32_t(q & 3) * 4u;
    // this lane's part of the B fragments (the other lanes read the zeros)
    const uint32_t lane_x1 = (q >> 1) == t ? uint32_t(q) * 8u : 96u;
    const uint32_t lane_x2 = q == 2 * t ? 64u + uint32_t(t) * 8u : 96u;
    const uint32_t lane_xs = 104u + 4u * uint32_t(t);
    const uint32_t cp0_gp = uint32_t(lane >> 2), cp1_gp = 8u + uint32_t(lane >> 2), cp_col = uint32_t(lane & 3);
    const uint32_t cp0_dst = (cp0_gp / 3u) * kBatRingGroup + (cp0_gp % 3u) * 64u + cp_col * 16u;
    const uint32_t cp1_dst = (cp1_gp / 3u) * kBatRingGroup + (cp1_gp % 3u) * 64u + cp_col * 16u;

    const uint32_t ctas = gridDim.x, cells = uint32_t(tile_groups) * uint32_t(col_groups), CG = uint32_t(col_groups);
    const uint32_t cell_begin = uint32_t(uint64_t(blockIdx.x) * cells / ctas);
    const uint32_t cell_end = uint32_t((uint64_t(blockIdx.x) + 1) * cells / ctas);
    uint32_t tg = cell_begin / CG, cg = cell_begin - tg * CG;

    auto fetch = [&](uint32_t ftg, uint32_t fcg, uint32_t slot) {
        const uint32_t G0 = (ftg * kBatWarps + uint32_t(warp)) * (2 * RB);
        const uint32_t col = fcg * PC + cp_col;
        const bool in = col < Bu;
        const uint4* base = reinterpret_cast<const uint4*>(codes) + size_t(G0) * 3 * Bu + (in ? col : 0u);
        const uint32_t dst = ring + slot * kBatRingSlot;
        const bool have0 = in && G0 + cp0_gp / 3u < uint32_t(row_groups);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst + cp0_dst),
                     "l"(have0 ? base + size_t(cp0_gp) * Bu : reinterpret_cast<const uint4*>(codes)), "r"(have0 ? 16u : 0u));
        if (lane < 16) {
            const bool have1 = in && G0 + cp1_gp / 3u < uint32_t(row_groups);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst + cp1_dst),
                         "l"(have1 ? base + size_t(cp1_gp) * Bu : reinterpret_cast<const uint4*>(codes)), "r"(have1 ? 16u : 0u));
        }
        asm volatile("cp.async.commit_group;");
    };
    if (cell_begin < cell_end) fetch(tg, cg, 0);
    else asm volatile("cp.async.commit_group;");
    pdl_wait();  // x may come from the preceding kernel; the partial results of an earlier call have been read

    // Image of a chunk of CP passes: thread (pass i, column cs, vector v) quantises one column of one vector and
    // writes its planes into the quad's record as B fragments.
    auto image_build = [&](uint32_t first_cell) {
        for (int id = threadIdx.x; id < CP * PC * V; id += kBatThreads) {
            const int v = id % V, cs = (id / V) % PC, i = id / (V * PC);
            const uint32_t cell = first_cell + uint32_t(i);
            if (cell >= cell_end) continue;
            const int col = int(cell % CG) * PC + cs;
            uint32_t qv[20];
            if (col < B) {
                quantise_column(x + size_t(v) * K, K, col, qv);
            } else {
#pragma unroll
                for (int k = 0; k < 20; ++k) qv[k] = 0u;
            }
            unsigned char* rec = image_ptr + size_t(i * V + v) * kQuadBytes;
#pragma unroll
            for (int pr = 0; pr < 3; ++pr) {
                unsigned char* line = rec + 128 * pr;
                *reinterpret_cast<uint2*>(line + 16 * cs) = make_uint2(qv[6 + 2 * pr], qv[7 + 2 * pr]);        // middle plane
                *reinterpret_cast<uint2*>(line + 16 * cs + 8) = make_uint2(qv[12 + 2 * pr], qv[13 + 2 * pr]);  // low plane
                *reinterpret_cast<uint2*>(line + 64 + 8 * cs) = make_uint2(qv[2 * pr], qv[2 * pr + 1]);        // high plane
                if (cs == 0) *reinterpret_cast<uint2*>(line + 96) = make_uint2(0u, 0u);
            }
            *reinterpret_cast<uint32_t*>(rec + 104 + 4 * cs) = qv[18];
        }
    };
    image_build(cell_begin);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();  // tables staged, first image built

    float acc[RB][2][V];
#pragma unroll
    for (int rb = 0; rb < RB; ++rb)
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int v = 0; v < V; ++v) acc[rb][j][v] = 0.f;

    for (uint32_t cell = cell_begin; cell < cell_end; ++cell) {
        const uint32_t pass = cell - cell_begin, slot = pass & 1u, in_chunk = pass % CP;
        const bool active = (int(tg) * kBatWarps + warp) * (16 * RB) < N;  // warp-uniform
        uint32_t ntg = tg, ncg = cg + 1;
        if (ncg == CG) { ncg = 0; ++ntg; }
        if (in_chunk == 0 && pass > 0) {  // CTA-uniform: the image of the next chunk of passes replaces the old one
            __syncthreads();
            image_build(cell);
            __syncthreads();
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();  // every lane's copies have landed, and every lane has left the other slot
        if (cell + 1 < cell_end) fetch(ntg, ncg, slot ^ 1u);
        if (active) {
            const uint32_t src = ring + slot * kBatRingSlot;
            FastBlock f[RB][2];
            float scale[RB][2];
#pragma unroll
            for (int rb = 0; rb < RB; ++rb) {
                uint2 w0;
                uint32_t w1pair;
                asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(w0.x), "=r"(w0.y) : "r"(src + lane_w0 + rb * 2 * kBatRingGroup));
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w1pair) : "r"(src + lane_w1 + rb * 2 * kBatRingGroup));
                fast_decode<false>(sm_tab, w0.x, w1pair, f[rb][0]);
                fast_decode<true>(sm_tab, w0.y, w1pair, f[rb][1]);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    int n2 = int(f[rb][j].goff);
#pragma unroll
                    for (int k = 0; k < 6; ++k) n2 = dp4a_ss(f[rb][j].y[k], f[rb][j].y[k], n2);
                    scale[rb][j] = lds32f(uint32_t(n2));
                }
            }
            const uint32_t img = image + in_chunk * (V * kQuadBytes);
#pragma unroll
            for (int v = 0; v < V; ++v) {
                uint2 bm[3], bh[3];
#pragma unroll
                for (int pr = 0; pr < 3; ++pr) {
                    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(bm[pr].x), "=r"(bm[pr].y) : "r"(img + v * kQuadBytes + 128 * pr + lane_x1));
                    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(bh[pr].x), "=r"(bh[pr].y) : "r"(img + v * kQuadBytes + 128 * pr + lane_x2));
                }
                float step;
                asm volatile("ld.shared.f32 %0, [%1];" : "=f"(step) : "r"(img + v * kQuadBytes + lane_xs));
                if constexpr (V <= 2) {  // registers allow the two row blocks' MMA chains side by side
                int dm[RB][4], dh[RB][4];
#pragma unroll
                for (int rb = 0; rb < RB; ++rb)
#pragma unroll
                    for (int i = 0; i < 4; ++i) { dm[rb][i] = 0; dh[rb][i] = 0; }
#pragma unroll
                for (int pr = 0; pr < 3; ++pr)
#pragma unroll
                    for (int rb = 0; rb < RB; ++rb) {
                        mma_bd(dm[rb], f[rb][0].y[2 * pr], f[rb][1].y[2 * pr], f[rb][0].y[2 * pr + 1], f[rb][1].y[2 * pr + 1],
                               bm[pr].x, bm[pr].y, dm[rb], false);
                        mma_bd(dh[rb], f[rb][0].y[2 * pr], f[rb][1].y[2 * pr], f[rb][0].y[2 * pr + 1], f[rb][1].y[2 * pr + 1],
                               bh[pr].x, bh[pr].y, dh[rb], true);
                    }
#pragma unroll
                for (int rb = 0; rb < RB; ++rb) {
                    const int dot0 = dh[rb][0] * 65536 + (dm[rb][0] * 256 + dm[rb][1]);
                    const int dot1 = dh[rb][2] * 65536 + (dm[rb][2] * 256 + dm[rb][3]);
                    acc[rb][0][v] = fmaf(float(dot0), scale[rb][0] * step, acc[rb][0][v]);
                    acc[rb][1][v] = fmaf(float(dot1), scale[rb][1] * step, acc[rb][1][v]);
                }
                } else {
#pragma unroll
                for (int rb = 0; rb < RB; ++rb) {
                    int dm[4] = {0, 0, 0, 0}, dh[4] = {0, 0, 0, 0};
#pragma unroll
                    for (int pr = 0; pr < 3; ++pr) {
                        mma_bd(dm, f[rb][0].y[2 * pr], f[rb][1].y[2 * pr], f[rb][0].y[2 * pr + 1], f[rb][1].y[2 * pr + 1],
                               bm[pr].x, bm[pr].y, dm, false);
                        mma_bd(dh, f[rb][0].y[2 * pr], f[rb][1].y[2 * pr], f[rb][0].y[2 * pr + 1], f[rb][1].y[2 * pr + 1],
                               bh[pr].x, bh[pr].y, dh, true);
                    }
                    // exact int32 dot products of -y with the 24-bit activations (the scale carries the other minus sign)
                    const int dot0 = dh[0] * 65536 + (dm[0] * 256 + dm[1]);
                    const int dot1 = dh[2] * 65536 + (dm[2] * 256 + dm[3]);
                    acc[rb][0][v] = fmaf(float(dot0), scale[rb][0] * step, acc[rb][0][v]);
                    acc[rb][1][v] = fmaf(float(dot1), scale[rb][1] * step, acc[rb][1][v]);
                }
                }
            }
        }
        if (cell + 1 == cell_end || ntg != tg) {  // CTA-uniform: this CTA's piece of tile group tg is complete
            // the four lanes of a row (its four columns) are added, then lane t = 0 writes the row's V sums
            float* mine = partials + (size_t(blockIdx.x + tg) * kBatWarps + warp) * kPieceFloats;
#pragma unroll
            for (int rb = 0; rb < RB; ++rb)
#pragma unroll
                for (int j = 0; j < 2; ++j)
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        float sum = acc[rb][j][v];
                        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
                        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
                        if (t == 0) mine[(16 * rb + 2 * q + j) * 8 + v] = sum;
                        acc[rb][j][v] = 0.f;
                    }
        }
        tg = ntg;
        cg = ncg;
    }
}

// Sum of a tile group's pieces in CTA order, row scale, tail (Sec. 5.1): one thread per (row, vector).
template <int NG, int RB>
__global__ void __launch_bounds__(256)
k_combine_batched(const float* __restrict__ partials, const float* __restrict__ row_scales,
                  const __half* __restrict__ x, const __half* __restrict__ tail, float* __restrict__ y, int N, int K,
                  int B, int batch, int tile_groups, int col_groups, int ctas) {
    constexpr int kPieceFloats = RB * 128 * NG, kGroupRows = kBatWarps * 16 * RB;
    pdl_release();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int v = idx % (8 * NG), r = idx / (8 * NG);
    const bool mine = r < N && v < batch;
    // what does not depend on the pieces comes before the wait for k_gemv_batched
    const int rr = mine ? r : 0;
    const uint32_t tg = uint32_t(rr / kGroupRows), CG = uint32_t(col_groups);
    const int warp = (rr % kGroupRows) / (16 * RB), rt = rr % (16 * RB);
    const uint32_t cells = uint32_t(tile_groups) * CG;
    const uint32_t first = cta_of_cell(tg * CG, uint32_t(ctas), cells);
    const uint32_t pieces = cta_of_cell(tg * CG + CG - 1, uint32_t(ctas), cells) - first + 1;
    const float scale = mine ? __ldg(row_scales + r) : 0.f;
    pdl_wait();  // the pieces come from k_gemv_batched
    if (!mine) return;
    const float* p = partials + (size_t(first + tg) * kBatWarps + warp) * kPieceFloats + rt * (8 * NG) + v;
    // sixteen pieces are loaded at a time (all of them, for the usual split of a tile group over about twenty
    // CTAs, in two rounds of independent loads) and added in piece order
    float total = 0.f;
    for (uint32_t k0 = 0; k0 < pieces; k0 += 16) {
        float v[16];
#pragma unroll
        for (uint32_t j = 0; j < 16; ++j) v[j] = k0 + j < pieces ? __ldcg(p + size_t(k0 + j) * kBatWarps * kPieceFloats) : 0.f;
#pragma unroll
        for (uint32_t j = 0; j < 16; ++j) total += v[j];
    }
    float res = scale * total;
    const int ntail = tail ? K % 24 : 0;
    for (int k = 0; k < ntail; ++k)
        res = fmaf(__half2float(tail[size_t(r) * ntail + k]), __half2float(x[size_t(v) * K + 24 * B + k]), res);
    y[size_t(v) * N + r] = res;
}

// Scratch: partial results, one piece per (CTA, tile group) pair that occurs.
struct BatchedPlan {
    int tile_groups, col_groups, ctas;
    size_t total;
};
static BatchedPlan batched_plan(int N, int B, int rb, int max_ctas) {
    BatchedPlan P;
    const int pc = kPassTiles / rb, group_rows = kBatWarps * 16 * rb;
    P.tile_groups = (N + group_rows - 1) / group_rows;
    P.col_groups = (B + pc - 1) / pc;
    const long long cells = (long long)P.tile_groups * P.col_groups;
    P.ctas = int(cells < max_ctas ? cells : max_ctas);
    if (P.ctas < 1) P.ctas = 1;
    P.total = size_t(P.ctas + P.tile_groups) * kBatWarps * (size_t(rb) * 256) * 4;  // sized for two vector groups
    return P;
}

// Row blocks per warp for a batch size.
static int batched_rb(int batch) { return batch <= 8 ? TETRA_BAT_RB1 : TETRA_BAT_RB2; }

// Upper bound over the grids this library launches (at most 1024 CTAs) and both kernel variants.
size_t batched_workspace_bytes(int N, int blocks_per_row) {
    const size_t a = batched_plan(N, blocks_per_row, batched_rb(1), 1024).total;
    const size_t b = batched_plan(N, blocks_per_row, batched_rb(16), 1024).total;
    return a > b ? a : b;
}

template <int NG, int RB>
static cudaError_t launch_variant(const void* codes, const float* row_scales, const void* table, const __half* xh,
                                  float* y, int N, int K, int B, int batch, const __half* tl, float* partials, int sms,
                                  uint32_t smem, cudaStream_t s) {
    const BatchedPlan P = batched_plan(N, B, RB, sms);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(P.ctas));
    cfg.blockDim = dim3(kBatThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_gemv_batched<NG, RB>, static_cast<const DeviceTables*>(table),
                                       static_cast<const unsigned char*>(codes), xh, N, K, B, batch, partials,
                                       P.tile_groups, P.col_groups);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cc = {};
    cc.gridDim = dim3(unsigned((size_t(N) * 8 * NG + 255) / 256));
    cc.blockDim = dim3(256);
    cc.stream = s;
    cc.attrs = attr;
    cc.numAttrs = 1;
    return cudaLaunchKernelEx(&cc, k_combine_batched<NG, RB>, static_cast<const float*>(partials), row_scales, xh, tl,
                              y, N, K, B, batch, P.tile_groups, P.col_groups, P.ctas);
}

template <int V>
static cudaError_t launch_few(const void* codes, const float* row_scales, const void* table, const __half* xh, float* y,
                              int N, int K, int B, const __half* tl, float* partials, int sms, cudaStream_t s) {
    const uint32_t smem = kTableSmemBytes + kBatWarps * 2 * kBatRingSlot + kFewChunkPasses * kFewMaxVectors * kQuadBytes;
    static PerDeviceOnce once;
    cudaError_t e = once.run([smem] { return cudaFuncSetAttribute(k_gemv_few<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)); });
    if (e != cudaSuccess) return e;
    const BatchedPlan P = batched_plan(N, B, 2, sms);
    e = launch_pdl(k_gemv_few<V>, P.ctas, kBatThreads, smem, s, static_cast<const DeviceTables*>(table),
                   static_cast<const unsigned char*>(codes), xh, N, K, B, partials, P.tile_groups, P.col_groups);
    if (e != cudaSuccess) return e;
    return launch_pdl(k_combine_batched<1, 2>, int((size_t(N) * 8 + 255) / 256), 256, 0, s, static_cast<const float*>(partials),
                      row_scales, xh, tl, y, N, K, B, V, P.tile_groups, P.col_groups, P.ctas);
}

cudaError_t launch_gemv_batched(const void* codes, const float* row_scales, const void* table, const void* x,
                                float* y, int N, int K, int batch, const void* tail, void* ws, cudaStream_t s) {
    int sms = 0;
    cudaError_t e = device_sms(&sms);
    if (e != cudaSuccess) return e;
    if (sms > 1024) sms = 1024;
    const uint32_t smem = kTableSmemBytes + kBatWarps * kBatWarpSmem + kImageGroups * kBatColBytesPerGroup;
    static PerDeviceOnce once;
    e = once.run([smem] {
        cudaError_t r = cudaFuncSetAttribute(k_gemv_batched<1, TETRA_BAT_RB1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (r == cudaSuccess)
            r = cudaFuncSetAttribute(k_gemv_batched<2, TETRA_BAT_RB2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        return r;
    });
    if (e != cudaSuccess) return e;
    const int B = tail ? K / 24 : (K + 23) / 24;
    const __half* xh = static_cast<const __half*>(x);
    const __half* tl = static_cast<const __half*>(tail);
    float* partials = static_cast<float*>(ws);
#ifndef TETRA_NO_FEW
    if (batch == 2) return launch_few<2>(codes, row_scales, table, xh, y, N, K, B, tl, partials, sms, s);
    if (batch == 3) return launch_few<3>(codes, row_scales, table, xh, y, N, K, B, tl, partials, sms, s);
    if (batch == 4) return launch_few<4>(codes, row_scales, table, xh, y, N, K, B, tl, partials, sms, s);
#endif
    if (batch <= 8)
        return launch_variant<1, TETRA_BAT_RB1>(codes, row_scales, table, xh, y, N, K, B, batch, tl, partials, sms, smem, s);
    return launch_variant<2, TETRA_BAT_RB2>(codes, row_scales, table, xh, y, N, K, B, batch, tl, partials, sms, smem, s);
}

}  // namespace tetra
