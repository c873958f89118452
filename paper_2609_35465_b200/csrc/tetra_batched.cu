// Decode-and-multiply for 2..16 activation vectors at once (Eq. (2), Sec. 5.1).
//
// A block is decoded once and multiplied with every vector, so the decode cost
// is shared.  The products over a block's 24 coordinates for up to 16 vectors
// are a small dense contraction, int8 x int8 -> int32, and run on the tensor
// cores (mma.sync m16n8k32); everything around it (field extraction, table
// lookups, per-block scale, FP32 accumulation) is the batch-1 decoder.
//
// Thread layout: a warp owns a tile of 16 rows and walks a chunk of the block
// columns eight at a time.  In one pass lane l decodes four blocks (row l % 16,
// columns l / 16 + 2 j), writes each block's 24 int8 coordinates as one 32-byte
// row of a 16 x 32 shared-memory tile (coordinates 24..31 are zero) and the
// block's scale next to it; the warp then loads the tiles as MMA A fragments with
// ldmatrix and multiplies them with the three int8 planes of the activations'
// 24-bit fixed-point image (B fragments, read from the scratch area).  The
// int32 results of the planes are combined exactly, converted once, scaled by
// block scale x activation step and added into FP32 accumulators that the lane
// keeps for its (row, vector) pairs: no cross-lane reduction is needed.
#include <cuda_fp16.h>

#include "tetra_device.cuh"
#include "tetra_launch.h"

namespace tetra {

constexpr int kBatThreads = 512;
constexpr int kBatWarps = kBatThreads / 32;
constexpr int kBatMax = 16;
// Scratch per block column: planes [3][8 words][16 vectors] (words 6, 7 and unused vectors zero), then 16 steps.
constexpr int kBatColWords = 3 * 8 * 16 + 16;
constexpr int kBatColBytes = kBatColWords * 4;

// One thread per (block column, vector): the 24-bit fixed-point image of 24 activations, scattered
// into the layout the B fragments are read from.
__global__ void __launch_bounds__(256) k_prepare_batched(const __half* __restrict__ x, int K, int B, int batch,
                                                         uint32_t* __restrict__ xqb, int32_t* __restrict__ counters,
                                                         int tiles) {
    pdl_release();
    pdl_wait();
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < tiles; t += gridDim.x * blockDim.x) counters[t] = 0;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < B * kBatMax; t += gridDim.x * blockDim.x) {
        const int c = t / kBatMax, v = t % kBatMax;
        uint32_t q[20];
        if (v < batch) {
            quantise_column(x + size_t(v) * K, K, c, q);
        } else {
#pragma unroll
            for (int k = 0; k < 20; ++k) q[k] = 0;
        }
        uint32_t* col = xqb + size_t(c) * kBatColWords;
#pragma unroll
        for (int pl = 0; pl < 3; ++pl)
#pragma unroll
            for (int w = 0; w < 8; ++w) col[(pl * 8 + w) * 16 + v] = w < 6 ? q[pl * 6 + w] : 0u;
        col[3 * 8 * 16 + v] = q[18];  // the step (float bits); 0 for unused vectors
    }
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

constexpr int kPassCols = 8;                                   // block columns per pass (four blocks per lane)
constexpr int kBatWarpSmem = kPassCols * 512 + kPassCols * 64;  // coordinate tiles + block scales

// B fragments (three planes) and steps of one block column for this lane.
template <int NG>
struct ColumnB {
    uint32_t b[NG][3][2];
    float2 step[NG];
};
template <int NG>
__device__ __forceinline__ void load_column_b(const uint32_t* __restrict__ xc, int g, int t4, ColumnB<NG>& C) {
#pragma unroll
    for (int n = 0; n < NG; ++n) {
        const uint32_t* bp = xc + 8 * n + g;  // words t4 and 4 + t4 of vector 8 n + g
#pragma unroll
        for (int pl = 0; pl < 3; ++pl) {
            C.b[n][pl][0] = __ldg(bp + (pl * 8 + t4) * 16);
            C.b[n][pl][1] = __ldg(bp + (pl * 8 + 4 + t4) * 16);
        }
        C.step[n] = __ldg(reinterpret_cast<const float2*>(xc + 3 * 8 * 16 + 8 * n + 2 * t4));
    }
}

template <int NG>  // vector groups of eight: 1 (batch <= 8) or 2
__global__ void __launch_bounds__(kBatThreads, 1)
k_gemv_batched(const DeviceTables* __restrict__ tab, const unsigned char* __restrict__ codes,
               const float* __restrict__ row_scales, const __half* __restrict__ x, const __half* __restrict__ tail,
               float* __restrict__ y, int N, int K, int B, int batch, const uint32_t* __restrict__ xqb,
               int32_t* __restrict__ counters, float* __restrict__ partials, int chunks, int chunk_cols) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pdl_release();
    unsigned char* smem = stage_fast_tables(tab, smem_raw);
    const uint32_t sm_tab = smem_u32(smem);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // per warp: eight 16 x 32-byte tiles of coordinates (one per block column of a pass), then 8 x 16 block scales
    unsigned char* tiles = smem + kFastBytes + warp * kBatWarpSmem;
    float* scales = reinterpret_cast<float*>(tiles + kPassCols * 512);
    const int row16 = lane & 15, colsel = lane >> 4;
#pragma unroll
    for (int j = 0; j < 4; ++j)  // coordinates 24..31 of every tile row stay zero for the whole kernel
        *reinterpret_cast<uint2*>(tiles + (colsel + 2 * j) * 512 + row16 * 32 + 24) = make_uint2(0u, 0u);
    __syncthreads();
    pdl_wait();  // the activation image comes from k_prepare_batched

    const int rows_padded = ((N + 7) / 8) * 8;
    const int tiles_total = (N + 15) / 16;
    const uint32_t Bu = uint32_t(B);
    const int g = lane >> 2, t4 = lane & 3;  // MMA fragment coordinates
    const uint32_t tile_addr = smem_u32(tiles);
    // ldmatrix: lane provides the address of row (lane % 8) of 8x8 matrix (lane / 8):
    // matrices = (rows 0-7, bytes 0-15), (rows 8-15, bytes 0-15), (rows 0-7, bytes 16-31), (rows 8-15, bytes 16-31)
    const uint32_t ldm_off = uint32_t((((lane >> 3) & 1) * 8 + (lane & 7)) * 32 + (lane >> 4) * 16);

    // A unit is a 16-row tile x a chunk of the block columns (chunk_cols is a multiple of 8); the chunks of
    // a tile leave their 16 x 16 partial results in the scratch area and the last one to arrive adds them
    // up in chunk order (fixed order, no waiting, no floating-point atomics).
    const int units_total = tiles_total * chunks;
    for (int unit = blockIdx.x * kBatWarps + warp; unit < units_total; unit += gridDim.x * kBatWarps) {
        const int tile = unit / chunks, chunk = unit - tile * chunks;
        const uint32_t c_begin = uint32_t(chunk) * uint32_t(chunk_cols);
        const uint32_t c_end = min(Bu, c_begin + uint32_t(chunk_cols));
        const int row = tile * 16 + row16;
        float acc[NG][4];
#pragma unroll
        for (int n = 0; n < NG; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[n][i] = 0.f;
        // lane (row16, colsel) decodes columns c0 + colsel + 2 j, j = 0..3, of each pass
        uint32_t w0[4], w1[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            load_block_words(codes, c_end, row, rows_padded, c_begin + colsel + 2 * j, Bu, &w0[j], &w1[j]);
        for (uint32_t c0 = c_begin; c0 < c_end; c0 += kPassCols) {
            uint32_t cw0[4], cw1[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) { cw0[j] = w0[j]; cw1[j] = w1[j]; }
#pragma unroll
            for (int j = 0; j < 4; ++j)  // next pass
                load_block_words(codes, c_end, row, rows_padded, c0 + kPassCols + colsel + 2 * j, Bu, &w0[j], &w1[j]);
            ColumnB<NG> cur;
            load_column_b<NG>(xqb + size_t(c0) * kBatColWords, g, t4, cur);  // in flight during the decode
            __syncwarp();  // the previous pass's fragments have been read
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                FastBlock fb;
                fast_decode<false>(sm_tab, cw0[j], cw1[j], fb);
                int n2 = 0;
#pragma unroll
                for (int k = 0; k < 6; ++k) n2 = dp4a_ss(fb.y[k], fb.y[k], n2);
                const float scale = lds32f(fb.goff | ((uint32_t(n2) >> 2) & 0x7Cu));  // gain[g] / sqrt(16 m)
                uint2* dst = reinterpret_cast<uint2*>(tiles + (colsel + 2 * j) * 512 + row16 * 32);
                dst[0] = make_uint2(fb.y[0], fb.y[1]);
                dst[1] = make_uint2(fb.y[2], fb.y[3]);
                dst[2] = make_uint2(fb.y[4], fb.y[5]);
                scales[(colsel + 2 * j) * 16 + row16] = scale;
            }
            __syncwarp();
#pragma unroll
            for (int cs = 0; cs < kPassCols; ++cs) {
                const uint32_t col = c0 + cs;
                if (col < c_end) {  // warp-uniform
                    ColumnB<NG> nxt;
                    if (cs + 1 < kPassCols && col + 1 < c_end)
                        load_column_b<NG>(xqb + size_t(col + 1) * kBatColWords, g, t4, nxt);
                    uint32_t a[4];
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                                 : "r"(tile_addr + cs * 512 + ldm_off));
                    const float s_lo = scales[cs * 16 + g], s_hi = scales[cs * 16 + g + 8];
#pragma unroll
                    for (int n = 0; n < NG; ++n) {
                        int dh[4], dm[4], dl[4];
                        mma_s8s8(dh, a, cur.b[n][0][0], cur.b[n][0][1]);
                        mma_s8u8(dm, a, cur.b[n][1][0], cur.b[n][1][1]);
                        mma_s8u8(dl, a, cur.b[n][2][0], cur.b[n][2][1]);
                        // this lane's results: rows g (i = 0, 1) and g + 8 (i = 2, 3), vectors 8 n + 2 t4 + (i & 1)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int dot = dh[i] * 65536 + (dm[i] * 256 + dl[i]);  // exact: |dot| < 2^31
                            acc[n][i] = fmaf(float(dot), (i < 2 ? s_lo : s_hi) * ((i & 1) ? cur.step[n].y : cur.step[n].x),
                                             acc[n][i]);
                        }
                    }
                    if (cs + 1 < kPassCols) cur = nxt;
                }
            }
        }
        // this lane's 4 NG results go to the tile's partial buffer of this chunk: [chunk][row 0..15][vector 0..15]
        float* mine = partials + (size_t(tile) * chunks + chunk) * 256;
#pragma unroll
        for (int n = 0; n < NG; ++n)
#pragma unroll
            for (int i = 0; i < 4; i += 2)
                *reinterpret_cast<float2*>(mine + (g + (i < 2 ? 0 : 8)) * 16 + 8 * n + 2 * t4) =
                    make_float2(acc[n][i], acc[n][i + 1]);
        __threadfence();
        __syncwarp();
        int arrived = 0;
        if (lane == 0) arrived = atomicAdd(counters + tile, 1);
        arrived = __shfl_sync(0xFFFFFFFFu, arrived, 0);
        if (arrived == chunks - 1) {  // all chunks of the tile are in: chunk-ordered sum, row scale, tail (Sec. 5.1)
            __threadfence();
            const int ntail = tail ? K % 24 : 0;
            const float* all = partials + size_t(tile) * chunks * 256;
#pragma unroll
            for (int n = 0; n < NG; ++n)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r16 = g + (i < 2 ? 0 : 8), r = tile * 16 + r16;
                    const int v = 8 * n + 2 * t4 + (i & 1);
                    if (r < N && v < batch) {
                        float total = 0.f;
                        for (int k = 0; k < chunks; ++k) total += __ldcg(all + size_t(k) * 256 + r16 * 16 + v);
                        float res = __ldg(row_scales + r) * total;
                        for (int k = 0; k < ntail; ++k)
                            res = fmaf(__half2float(tail[size_t(r) * ntail + k]),
                                       __half2float(x[size_t(v) * K + 24 * B + k]), res);
                        y[size_t(v) * N + r] = res;
                    }
                }
        }
    }
}

// Scratch: activation image | arrival counters (one per 16-row tile) | partial results.
struct BatchedPlan {
    int tiles, chunks, chunk_cols;
    size_t off_counters, off_partials, total;
};
static BatchedPlan batched_plan(int N, int B, int warps) {
    BatchedPlan P;
    P.tiles = (N + 15) / 16;
    int chunks = (2 * warps + P.tiles - 1) / P.tiles;        // about two units per warp
    if (chunks < 1) chunks = 1;
    int cols = (B + chunks - 1) / chunks;
    cols = (cols + kPassCols - 1) / kPassCols * kPassCols;     // passes take eight columns
    P.chunk_cols = cols;
    P.chunks = (B + cols - 1) / cols;
    P.off_counters = (size_t(B) * kBatColBytes + 255) & ~size_t(255);
    P.off_partials = (P.off_counters + size_t(P.tiles) * 4 + 255) & ~size_t(255);
    P.total = P.off_partials + size_t(P.tiles) * P.chunks * 256 * 4;
    return P;
}

// Upper bound over the grids this library launches (at most 8192 warps).
size_t batched_workspace_bytes(int N, int blocks_per_row) { return batched_plan(N, blocks_per_row, 8192).total; }

cudaError_t launch_gemv_batched(const void* codes, const float* row_scales, const void* table, const void* x,
                                float* y, int N, int K, int batch, const void* tail, void* ws, cudaStream_t s) {
    static bool attr_set[64] = {false};
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const uint32_t smem = kTableSmemBytes + kBatWarps * kBatWarpSmem;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(k_gemv_batched<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(k_gemv_batched<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int B = tail ? K / 24 : (K + 23) / 24;
    const __half* xh = static_cast<const __half*>(x);
    uint32_t* xqb = static_cast<uint32_t*>(ws);
    const BatchedPlan P = batched_plan(N, B, sms * kBatWarps);
    int32_t* counters = reinterpret_cast<int32_t*>(static_cast<unsigned char*>(ws) + P.off_counters);
    float* partials = reinterpret_cast<float*>(static_cast<unsigned char*>(ws) + P.off_partials);
    k_prepare_batched<<<sms * 2, 256, 0, s>>>(xh, K, B, batch, xqb, counters, P.tiles);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int units = P.tiles * P.chunks;
    int grid = (units + kBatWarps - 1) / kBatWarps;
    if (grid > sms) grid = sms;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid));
    cfg.blockDim = dim3(kBatThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const DeviceTables* tb = static_cast<const DeviceTables*>(table);
    const unsigned char* cd = static_cast<const unsigned char*>(codes);
    const __half* tl = static_cast<const __half*>(tail);
    if (batch <= 8)
        return cudaLaunchKernelEx(&cfg, k_gemv_batched<1>, tb, cd, row_scales, xh, tl, y, N, K, B, batch,
                                  static_cast<const uint32_t*>(xqb), counters, partials, P.chunks, P.chunk_cols);
    return cudaLaunchKernelEx(&cfg, k_gemv_batched<2>, tb, cd, row_scales, xh, tl, y, N, K, B, batch,
                              static_cast<const uint32_t*>(xqb), counters, partials, P.chunks, P.chunk_cols);
}

}  // namespace tetra
