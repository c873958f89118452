// Decode-and-multiply for 2..16 activation vectors at once (Eq. (2), Sec. 5.1).
//
// A block is decoded once and multiplied with every vector, so the decode cost
// is shared.  The products over a block's 24 coordinates for up to 16 vectors
// are a small dense contraction, int8 x int8 -> int32, and run on the tensor
// cores (mma.sync m16n8k32); everything around it (field extraction, table
// lookups, per-block scale, FP32 accumulation) is the batch-1 decoder.
//
// Thread layout: a warp owns RB row blocks of 16 rows, a CTA of 16 warps a group of 16 such row tiles,
// and the CTA walks the block columns 8 / RB at a time; such a (tile group, column group) cell is the
// unit of work, and the CTAs take equal contiguous ranges of the tile-group-major cell order.  In one
// pass lane l decodes four blocks (row l % 16 of row block j % RB, column l / 16 + 2 (j / RB), j = 0..3),
// writes each block's 24 int8 coordinates as a row of a shared-memory tile (coordinates 24..31 are zero)
// and the block's scale next to it; the warp then loads the tiles as MMA A fragments with ldmatrix and
// multiplies them with the three int8 planes of the activations' 24-bit fixed-point image (B fragments,
// read once per column and used for the warp's RB row blocks).  The image of a pass's columns is built
// by the CTA itself, in shared memory, during the pass before.  The int32 results of the planes are
// combined exactly, converted once, scaled by block scale x activation step and added into FP32
// accumulators that the lane keeps for its (row, vector) pairs: no cross-lane reduction is needed.  When a
// CTA's range leaves a tile group, its partial sums go to the scratch area as one piece; a second, small
// kernel adds the pieces of every tile group in CTA order (fixed order, no atomics, no flags), applies the
// row scale and the tail.  The only waits are CTA barriers and griddepcontrol.wait.
#include <cuda_fp16.h>

#include "tetra_device.cuh"
#include "tetra_launch.h"

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
// The image lives in shared memory only: the CTA builds the columns of its next pass while it works on the
// current one.
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

// Words of the block (row, col) from the packed layout; rows at or beyond rows_padded are the origin.
__device__ __forceinline__ void load_block_words(const unsigned char* __restrict__ codes, uint32_t col_end, int row,
                                                 int rows_padded, uint32_t col, uint32_t B, uint32_t* w0,
                                                 uint32_t* w1) {
    if (row >= rows_padded || col >= col_end) {
        *w0 = 0;
        *w1 = 0;
        return;
    }
    const uint32_t G = uint32_t(row) >> 3, r = uint32_t(row) & 7u;
    const unsigned char* rec = codes + (size_t(G) * 3 * B + col) * 16;
    *w0 = __ldg(reinterpret_cast<const uint32_t*>(rec + size_t(r >> 2) * B * 16 + (r & 3u) * 4));
    *w1 = __ldg(reinterpret_cast<const unsigned short*>(rec + size_t(2) * B * 16 + r * 2));
}

constexpr int kTileRow = 48;                // bytes per tile row: 24 coordinates, 8 zeros, 16 pad
constexpr int kTileBytes = 16 * kTileRow;   // (48-byte rows keep ldmatrix and the tile stores conflict-free)
constexpr int kBatWarpSmem = kPassTiles * kTileBytes + kPassTiles * 64;  // coordinate tiles + block scales
constexpr int kBatColBytesPerGroup = kBatGroupWords * 4;                 // image of one column, per ng

__device__ __forceinline__ void lds128(uint32_t saddr, uint32_t (&v)[4]) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(saddr));
}

// CTA that owns cell x when CTA i owns cells [i * cells / ctas, (i + 1) * cells / ctas).
__device__ __forceinline__ uint32_t cta_of_cell(uint32_t x, uint32_t ctas, uint32_t cells) {
    return uint32_t(((uint64_t(x) + 1) * ctas - 1) / cells);
}

// NG: vector groups of eight, 1 (batch <= 8) or 2.  RB: 16-row blocks per warp.
template <int NG, int RB>
__global__ void __launch_bounds__(kBatThreads, 1)
k_gemv_batched(const DeviceTables* __restrict__ tab, const unsigned char* __restrict__ codes,
               const __half* __restrict__ x, int N, int K, int B, int batch, float* __restrict__ partials, int tile_groups, int col_groups) {
    constexpr int PC = kPassTiles / RB;  // block columns per pass
    constexpr int kSlotBytes = PC * NG * kBatColBytesPerGroup;
    constexpr int kPieceFloats = RB * 128 * NG;  // partial results of one warp: 16 RB rows x 8 NG vectors
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pdl_release();
    unsigned char* smem = stage_fast_tables(tab, smem_raw);
    const uint32_t sm_tab = smem_u32(smem);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // per warp: eight 16-row tiles of coordinates (tile rb * PC + column), then 8 x 16 block scales; after
    // the warps' areas, two slots for the activation image of a column group
    unsigned char* tiles = smem + kFastBytes + warp * kBatWarpSmem;
    float* scales = reinterpret_cast<float*>(tiles + kPassTiles * kTileBytes);
    const uint32_t slots = smem_u32(smem + kFastBytes + kBatWarps * kBatWarpSmem);
    const int row16 = lane & 15, colsel = lane >> 4;
#pragma unroll
    for (int j = 0; j < 4; ++j)  // coordinates 24..31 of every tile row stay zero for the whole kernel
        *reinterpret_cast<uint2*>(tiles + (colsel + 2 * j) * kTileBytes + row16 * kTileRow + 24) = make_uint2(0u, 0u);

    const int rows_padded = ((N + 7) / 8) * 8;
    const uint32_t Bu = uint32_t(B);
    const int g = lane >> 2, t4 = lane & 3;  // MMA fragment coordinates
    const uint32_t tile_addr = smem_u32(tiles);
    // ldmatrix: lane provides the address of row (lane % 8) of 8x8 matrix (lane / 8):
    // matrices = (rows 0-7, bytes 0-15), (rows 8-15, bytes 0-15), (rows 0-7, bytes 16-31), (rows 8-15, bytes 16-31)
    const uint32_t ldm_off = uint32_t((((lane >> 3) & 1) * 8 + (lane & 7)) * kTileRow + (lane >> 4) * 16);

    const uint32_t ctas = gridDim.x, cells = uint32_t(tile_groups) * uint32_t(col_groups), CG = uint32_t(col_groups);
    const uint32_t cell_begin = uint32_t(uint64_t(blockIdx.x) * cells / ctas);
    const uint32_t cell_end = uint32_t((uint64_t(blockIdx.x) + 1) * cells / ctas);
    uint32_t tg = cell_begin / CG, cg = cell_begin - tg * CG;

    // block j of the lane: row block j % RB, column colsel + 2 (j / RB) of the pass
    auto load_pass = [&](uint32_t group_tg, uint32_t group_cg, uint32_t (&w0)[4], uint32_t (&w1)[4]) {
        const int row0 = (int(group_tg) * kBatWarps + warp) * (16 * RB) + row16;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            load_block_words(codes, Bu, row0 + 16 * (j % RB), rows_padded, group_cg * PC + colsel + 2 * (j / RB), Bu,
                             &w0[j], &w1[j]);
    };
    uint32_t w0[4], w1[4];
    if (cell_begin < cell_end) load_pass(tg, cg, w0, w1);
    __syncthreads();
    pdl_wait();  // x may come from the preceding kernel; the partial results of an earlier call have been read
    // image tasks: warp w < PC * NG builds the group (column w / NG of the pass, vectors 8 (w % NG) + lane / 4)
    const bool image_warp = warp < PC * NG;
    const int image_col = warp / NG, image_vec = 8 * (warp % NG) + (lane >> 2);
    const uint32_t image_group = uint32_t(warp) * 1024u;
    ImageTask task;
    if (image_warp && cell_begin < cell_end) {
        image_load(x, K, batch, int(cg) * PC + image_col, image_vec, lane & 3, task);
        image_store(task, slots + image_group, image_vec, lane & 3);
    }

    float acc[RB][NG][4];
#pragma unroll
    for (int rb = 0; rb < RB; ++rb)
#pragma unroll
        for (int n = 0; n < NG; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[rb][n][i] = 0.f;

    for (uint32_t cell = cell_begin; cell < cell_end; ++cell) {
        const uint32_t slot = (cell - cell_begin) & 1u;
        const int row_base = (int(tg) * kBatWarps + warp) * (16 * RB);
        const bool active = row_base < N;  // warp-uniform
        uint32_t cw0[4], cw1[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { cw0[j] = w0[j]; cw1[j] = w1[j]; }
        uint32_t ntg = tg, ncg = cg + 1;
        if (ncg == CG) { ncg = 0; ++ntg; }
        __syncthreads();  // this cell's image is complete; everyone has left the slot the next one goes to
        const bool more = cell + 1 < cell_end;
        if (more) {
            if (image_warp) image_load(x, K, batch, int(ncg) * PC + image_col, image_vec, lane & 3, task);
            load_pass(ntg, ncg, w0, w1);
        }
        if (active) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                FastBlock fb;
                fast_decode<false>(sm_tab, cw0[j], cw1[j], fb);
                int n2 = 0;
#pragma unroll
                for (int k = 0; k < 6; ++k) n2 = dp4a_ss(fb.y[k], fb.y[k], n2);
                const float scale = lds32f(fb.goff | (uint32_t(n2) & 0x1F0u));  // gain[g] / sqrt(16 m)
                const int tile_id = (j % RB) * PC + 2 * (j / RB);  // + colsel
                unsigned char* dst = tiles + (tile_id + colsel) * kTileBytes + row16 * kTileRow;
                *reinterpret_cast<uint4*>(dst) = make_uint4(fb.y[0], fb.y[1], fb.y[2], fb.y[3]);
                *reinterpret_cast<uint2*>(dst + 16) = make_uint2(fb.y[4], fb.y[5]);
                scales[(tile_id + colsel) * 16 + row16] = scale;
            }
            __syncwarp();
            const uint32_t img = slots + slot * kSlotBytes + lane * 16;
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
                    const float s_lo = scales[tile_id * 16 + g], s_hi = scales[tile_id * 16 + g + 8];
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
        if (more && image_warp) image_store(task, slots + (slot ^ 1u) * kSlotBytes + image_group, image_vec, lane & 3);
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
    pdl_wait();  // the pieces come from k_gemv_batched
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int v = idx % (8 * NG), r = idx / (8 * NG);
    if (r >= N || v >= batch) return;
    const uint32_t tg = uint32_t(r / kGroupRows), CG = uint32_t(col_groups);
    const int warp = (r % kGroupRows) / (16 * RB), rt = r % (16 * RB);
    const uint32_t cells = uint32_t(tile_groups) * CG;
    const uint32_t first = cta_of_cell(tg * CG, uint32_t(ctas), cells);
    const uint32_t pieces = cta_of_cell(tg * CG + CG - 1, uint32_t(ctas), cells) - first + 1;
    const float* p = partials + (size_t(first + tg) * kBatWarps + warp) * kPieceFloats + rt * (8 * NG) + v;
    float total = 0.f;
#pragma unroll 8
    for (uint32_t k = 0; k < pieces; ++k) total += __ldcg(p + size_t(k) * kBatWarps * kPieceFloats);
    float res = __ldg(row_scales + r) * total;
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

cudaError_t launch_gemv_batched(const void* codes, const float* row_scales, const void* table, const void* x,
                                float* y, int N, int K, int batch, const void* tail, void* ws, cudaStream_t s) {
    int sms = 0;
    cudaError_t e = device_sms(&sms);
    if (e != cudaSuccess) return e;
    if (sms > 1024) sms = 1024;
    const uint32_t smem = kTableSmemBytes + kBatWarps * kBatWarpSmem + 2 * kPassTiles * 2 * kBatColBytesPerGroup;
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
    if (batch <= 8)
        return launch_variant<1, TETRA_BAT_RB1>(codes, row_scales, table, xh, y, N, K, B, batch, tl, partials, sms, smem, s);
    return launch_variant<2, TETRA_BAT_RB2>(codes, row_scales, table, xh, y, N, K, B, batch, tl, partials, sms, smem, s);
}

}  // namespace tetra
