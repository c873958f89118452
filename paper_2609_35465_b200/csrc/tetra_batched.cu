// Decode-and-multiply for 2..16 activation vectors at once (Eq. (2), Sec. 5.1).
//
// A block is decoded once and multiplied with every vector, so the decode cost
// is shared.  The products over a block's 24 coordinates for up to 16 vectors
// are a small dense contraction, int8 x int8 -> int32, and run on the tensor
// cores (mma.sync m16n8k32); everything around it (field extraction, table
// lookups, per-block scale, FP32 accumulation) is the batch-1 decoder.
//
// Thread layout: a CTA of 16 warps owns a group of 16 row tiles (warp w: 16 rows) and walks block columns
// eight at a time; such a (tile group, column group) cell is the unit of work, and the CTAs take equal
// contiguous ranges of the tile-group-major cell order.  In one pass lane l decodes four blocks (row l % 16,
// columns l / 16 + 2 j), writes each block's 24 int8 coordinates as a row of a shared-memory tile
// (coordinates 24..31 are zero) and the block's scale next to it; the warp then loads the tiles as MMA A
// fragments with ldmatrix and multiplies them with the three int8 planes of the activations' 24-bit
// fixed-point image (B fragments; the CTA copies the image of the next column group into shared memory
// with cp.async while it works on the current one).  The int32 results of the planes are combined exactly,
// converted once, scaled by block scale x activation step and added into FP32 accumulators that the lane
// keeps for its (row, vector) pairs: no cross-lane reduction is needed.  When a CTA's range leaves a tile
// group, its partial sums go to the scratch area; the last CTA to arrive at a tile group adds the pieces in
// CTA order (fixed order, no waiting, no floating-point atomics), applies the row scale and the tail.
#include <cuda_fp16.h>

#include "tetra_device.cuh"
#include "tetra_launch.h"

namespace tetra {

constexpr int kBatThreads = 512;
constexpr int kBatWarps = kBatThreads / 32;
constexpr int kBatMax = 16;
constexpr int kPassCols = 8;  // block columns per pass (four blocks per lane)
// Activation image per block column and vector group n (vectors 8 n .. 8 n + 7): two 16-byte chunks per
// lane, stored chunk-major ([chunk][lane][4 words]) so that a 128-bit access per chunk is contiguous over
// the warp:
//   chunk 2 n     = B-fragment registers (plane 0, h 0), (0, 1), (1, 0), (1, 1)
//   chunk 2 n + 1 = (2, 0), (2, 1), step of vector 8 n + 2 t, step of vector 8 n + 2 t + 1
// where the lane multiplies with vector 8 n + lane / 4, t = lane % 4, register h = 0 holds coordinates
// 4 t .. 4 t + 3 and h = 1 coordinates 16 + 4 t .. 16 + 4 t + 3 (24..31 and unused vectors are zero), and
// the steps are those of the lane's two result columns.  A column takes ng x 1 KiB (ng = 1 or 2 groups);
// the image covers the block columns rounded up to a multiple of eight (the extra ones are zero).
constexpr int kBatGroupWords = 2 * 32 * 4;

// One thread per (block column, vector, t): the 24-bit fixed-point image of the column's 24 activations,
// of which the thread stores the words of lane (vector % 8) * 4 + t, and two of the eight copies of the step.
__global__ void __launch_bounds__(256) k_prepare_batched(const __half* __restrict__ x, int K, int cols, int batch,
                                                         int ng, uint32_t* __restrict__ xqb,
                                                         int32_t* __restrict__ counters, int ncounters) {
    pdl_release();
    pdl_wait();
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < ncounters; t += gridDim.x * blockDim.x) counters[t] = 0;
    const int per_col = 32 * ng;  // (vector, t) pairs
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < cols * per_col; t += gridDim.x * blockDim.x) {
        const int c = t / per_col, v = (t % per_col) >> 2, tt = t & 3;
        uint32_t q[20];
        if (v < batch) {
            quantise_column(x + size_t(v) * K, K, c, q);
        } else {
#pragma unroll
            for (int k = 0; k < 20; ++k) q[k] = 0;
        }
        const int n = v >> 3, g = v & 7, ln = g * 4 + tt;
        uint32_t* grp = xqb + (size_t(c) * ng + n) * kBatGroupWords;
        uint32_t b[3][2];
#pragma unroll
        for (int pl = 0; pl < 3; ++pl) {
            // q[pl * 6 + k] holds coordinates 4 k .. 4 k + 3 of the plane
            uint32_t lo = q[pl * 6], hi = q[pl * 6 + 4];
            if (tt == 1) { lo = q[pl * 6 + 1]; hi = q[pl * 6 + 5]; }
            if (tt == 2) { lo = q[pl * 6 + 2]; hi = 0u; }
            if (tt == 3) { lo = q[pl * 6 + 3]; hi = 0u; }
            b[pl][0] = lo;
            b[pl][1] = hi;
        }
        *reinterpret_cast<uint4*>(grp + ln * 4) = make_uint4(b[0][0], b[0][1], b[1][0], b[1][1]);
        *reinterpret_cast<uint2*>(grp + (32 + ln) * 4) = make_uint2(b[2][0], b[2][1]);
        // the step goes to the eight lanes whose results belong to this vector: t = (v % 8) / 2, any g
#pragma unroll
        for (int gg = 2 * tt; gg < 2 * tt + 2; ++gg) grp[(32 + gg * 4 + (g >> 1)) * 4 + 2 + (v & 1)] = q[18];
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

constexpr int kTileRow = 48;                // bytes per tile row: 24 coordinates, 8 zeros, 16 pad
constexpr int kTileBytes = 16 * kTileRow;   // (48-byte rows keep ldmatrix and the tile stores conflict-free)
constexpr int kBatWarpSmem = kPassCols * kTileBytes + kPassCols * 64;  // coordinate tiles + block scales
constexpr int kBatSlotBytesPerGroup = kPassCols * kBatGroupWords * 4;  // image of one column group, per ng

__device__ __forceinline__ void lds128(uint32_t saddr, uint32_t (&v)[4]) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(saddr));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// CTA that owns cell x when CTA i owns cells [i * cells / ctas, (i + 1) * cells / ctas).
__device__ __forceinline__ uint32_t cta_of_cell(uint32_t x, uint32_t ctas, uint32_t cells) {
    return uint32_t(((uint64_t(x) + 1) * ctas - 1) / cells);
}

template <int NG>  // vector groups of eight: 1 (batch <= 8) or 2
__global__ void __launch_bounds__(kBatThreads, 1)
k_gemv_batched(const DeviceTables* __restrict__ tab, const unsigned char* __restrict__ codes,
               const float* __restrict__ row_scales, const __half* __restrict__ x, const __half* __restrict__ tail,
               float* __restrict__ y, int N, int K, int B, int batch, const uint32_t* __restrict__ xqb,
               int32_t* __restrict__ counters, float* __restrict__ partials, int tile_groups, int col_groups) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_last;
    pdl_release();
    unsigned char* smem = stage_fast_tables(tab, smem_raw);
    const uint32_t sm_tab = smem_u32(smem);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // per warp: eight 16-row tiles of coordinates (one per block column of a pass), then 8 x 16 block scales;
    // after the warps' areas, two slots for the activation image of a column group
    unsigned char* tiles = smem + kFastBytes + warp * kBatWarpSmem;
    float* scales = reinterpret_cast<float*>(tiles + kPassCols * kTileBytes);
    constexpr int kSlotBytes = NG * kBatSlotBytesPerGroup;
    const uint32_t slots = smem_u32(smem + kFastBytes + kBatWarps * kBatWarpSmem);
    const int row16 = lane & 15, colsel = lane >> 4;
#pragma unroll
    for (int j = 0; j < 4; ++j)  // coordinates 24..31 of every tile row stay zero for the whole kernel
        *reinterpret_cast<uint2*>(tiles + (colsel + 2 * j) * kTileBytes + row16 * kTileRow + 24) = make_uint2(0u, 0u);

    const int rows_padded = ((N + 7) / 8) * 8;
    const int tiles_total = (N + 15) / 16;
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

    // lane (row16, colsel) decodes columns 8 cg + colsel + 2 j, j = 0..3, of each pass
    uint32_t w0[4], w1[4];
    if (cell_begin < cell_end) {
        const int row = (int(tg) * kBatWarps + warp) * 16 + row16;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            load_block_words(codes, Bu, row, rows_padded, cg * kPassCols + colsel + 2 * j, Bu, &w0[j], &w1[j]);
    }
    __syncthreads();
    pdl_wait();  // the activation image comes from k_prepare_batched
    auto fetch_slot = [&](uint32_t group, uint32_t slot) {
        const unsigned char* src = reinterpret_cast<const unsigned char*>(xqb) + size_t(group) * kSlotBytes;
        for (int o = threadIdx.x * 16; o < kSlotBytes; o += kBatThreads * 16) cp_async16(slots + slot * kSlotBytes + o, src + o);
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if (cell_begin < cell_end) fetch_slot(cg, 0);

    float acc[NG][4];
#pragma unroll
    for (int n = 0; n < NG; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[n][i] = 0.f;

    for (uint32_t cell = cell_begin; cell < cell_end; ++cell) {
        const uint32_t slot = (cell - cell_begin) & 1u;
        const int tile = int(tg) * kBatWarps + warp;
        const bool active = tile < tiles_total;  // warp-uniform
        uint32_t cw0[4], cw1[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { cw0[j] = w0[j]; cw1[j] = w1[j]; }
        uint32_t ntg = tg, ncg = cg + 1;
        if (ncg == CG) { ncg = 0; ++ntg; }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();  // this cell's image has landed; everyone has left the slot the next copy overwrites
        if (cell + 1 < cell_end) {
            fetch_slot(ncg, slot ^ 1u);
            const int nrow = (int(ntg) * kBatWarps + warp) * 16 + row16;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                load_block_words(codes, Bu, nrow, rows_padded, ncg * kPassCols + colsel + 2 * j, Bu, &w0[j], &w1[j]);
        }
        if (active) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                FastBlock fb;
                fast_decode<false>(sm_tab, cw0[j], cw1[j], fb);
                int n2 = 0;
#pragma unroll
                for (int k = 0; k < 6; ++k) n2 = dp4a_ss(fb.y[k], fb.y[k], n2);
                const float scale = lds32f(fb.goff | ((uint32_t(n2) >> 2) & 0x7Cu));  // gain[g] / sqrt(16 m)
                unsigned char* dst = tiles + (colsel + 2 * j) * kTileBytes + row16 * kTileRow;
                *reinterpret_cast<uint4*>(dst) = make_uint4(fb.y[0], fb.y[1], fb.y[2], fb.y[3]);
                *reinterpret_cast<uint2*>(dst + 16) = make_uint2(fb.y[4], fb.y[5]);
                scales[(colsel + 2 * j) * 16 + row16] = scale;
            }
            __syncwarp();
            const uint32_t img = slots + slot * kSlotBytes + lane * 16;
#pragma unroll
            for (int cs = 0; cs < kPassCols; ++cs) {
                uint32_t a[4];
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                             : "r"(tile_addr + cs * kTileBytes + ldm_off));
                const float s_lo = scales[cs * 16 + g], s_hi = scales[cs * 16 + g + 8];
#pragma unroll
                for (int n = 0; n < NG; ++n) {
                    uint32_t q0[4], q1[4];
                    lds128(img + (cs * NG + n) * 1024, q0);
                    lds128(img + (cs * NG + n) * 1024 + 512, q1);
                    int dh[4], dm[4], dl[4];
                    mma_s8s8(dh, a, q0[0], q0[1]);
                    mma_s8u8(dm, a, q0[2], q0[3]);
                    mma_s8u8(dl, a, q1[0], q1[1]);
                    const float step_even = __uint_as_float(q1[2]), step_odd = __uint_as_float(q1[3]);
                    // this lane's results: rows g (i = 0, 1) and g + 8 (i = 2, 3), vectors 8 n + 2 t4 + (i & 1)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        int dot;  // dh * 65536 + dm * 256 + dl, exact (|dot| < 2^31), on the multiply-add pipe
                        asm("mad.lo.s32 %0, %1, 256, %2;" : "=r"(dot) : "r"(dm[i]), "r"(dl[i]));
                        asm("mad.lo.s32 %0, %1, 65536, %0;" : "+r"(dot) : "r"(dh[i]));
                        acc[n][i] = fmaf(float(dot), (i < 2 ? s_lo : s_hi) * ((i & 1) ? step_odd : step_even), acc[n][i]);
                    }
                }
            }
            __syncwarp();  // the fragments have been read before the next pass overwrites the tiles
        }
        if (cell + 1 == cell_end || ntg != tg) {  // CTA-uniform: this CTA's piece of tile group tg is complete
            // pieces are numbered blockIdx.x + tg: unique, and increasing along the cell order
            float* mine = partials + (size_t(blockIdx.x + tg) * kBatWarps + warp) * (128 * NG);
#pragma unroll
            for (int n = 0; n < NG; ++n)
#pragma unroll
                for (int i = 0; i < 4; i += 2) {
                    *reinterpret_cast<float2*>(mine + (g + (i < 2 ? 0 : 8)) * (8 * NG) + 8 * n + 2 * t4) =
                        make_float2(acc[n][i], acc[n][i + 1]);
                    acc[n][i] = 0.f;
                    acc[n][i + 1] = 0.f;
                }
            const uint32_t first = cta_of_cell(tg * CG, ctas, cells);
            const uint32_t pieces = cta_of_cell(tg * CG + CG - 1, ctas, cells) - first + 1;
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) s_last = atomicAdd(counters + tg, 1) == int(pieces) - 1;
            __syncthreads();
            if (s_last && active) {  // every piece of the tile group is in: ordered sum, row scale, tail (Sec. 5.1)
                __threadfence();
                const int ntail = tail ? K % 24 : 0;
                const float* all = partials + (size_t(first + tg) * kBatWarps + warp) * (128 * NG);
#pragma unroll
                for (int n = 0; n < NG; ++n)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int r16 = g + (i < 2 ? 0 : 8), r = tile * 16 + r16;
                        const int v = 8 * n + 2 * t4 + (i & 1);
                        if (r < N && v < batch) {
                            float total = 0.f;
                            for (uint32_t k = 0; k < pieces; ++k)
                                total += __ldcg(all + size_t(k) * kBatWarps * (128 * NG) + r16 * (8 * NG) + 8 * n + 2 * t4 + (i & 1));
                            float res = __ldg(row_scales + r) * total;
                            for (int k = 0; k < ntail; ++k)
                                res = fmaf(__half2float(tail[size_t(r) * ntail + k]),
                                           __half2float(x[size_t(v) * K + 24 * B + k]), res);
                            y[size_t(v) * N + r] = res;
                        }
                    }
            }
        }
        tg = ntg;
        cg = ncg;
    }
}

// Scratch: activation image | arrival counters (one per tile group) | partial results (one per piece).
struct BatchedPlan {
    int tile_groups, col_groups, ctas;
    size_t off_counters, off_partials, total;
};
static BatchedPlan batched_plan(int N, int B, int max_ctas) {
    BatchedPlan P;
    const int tiles = (N + 15) / 16;
    P.tile_groups = (tiles + kBatWarps - 1) / kBatWarps;
    P.col_groups = (B + kPassCols - 1) / kPassCols;
    const long long cells = (long long)P.tile_groups * P.col_groups;
    P.ctas = int(cells < max_ctas ? cells : max_ctas);
    if (P.ctas < 1) P.ctas = 1;
    P.off_counters = (size_t(P.col_groups) * 2 * kBatSlotBytesPerGroup + 255) & ~size_t(255);  // image for ng = 2
    P.off_partials = (P.off_counters + size_t(P.tile_groups) * 4 + 255) & ~size_t(255);
    P.total = P.off_partials + size_t(P.ctas + P.tile_groups) * kBatWarps * 256 * 4;
    return P;
}

// Upper bound over the grids this library launches (at most 1024 CTAs).
size_t batched_workspace_bytes(int N, int blocks_per_row) { return batched_plan(N, blocks_per_row, 1024).total; }

cudaError_t launch_gemv_batched(const void* codes, const float* row_scales, const void* table, const void* x,
                                float* y, int N, int K, int batch, const void* tail, void* ws, cudaStream_t s) {
    static bool attr_set[64] = {false};
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (sms > 1024) sms = 1024;
    const uint32_t smem = kTableSmemBytes + kBatWarps * kBatWarpSmem + 2 * 2 * kBatSlotBytesPerGroup;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(k_gemv_batched<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(k_gemv_batched<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int B = tail ? K / 24 : (K + 23) / 24;
    const int ng = batch <= 8 ? 1 : 2;
    const __half* xh = static_cast<const __half*>(x);
    uint32_t* xqb = static_cast<uint32_t*>(ws);
    const BatchedPlan P = batched_plan(N, B, sms);
    int32_t* counters = reinterpret_cast<int32_t*>(static_cast<unsigned char*>(ws) + P.off_counters);
    float* partials = reinterpret_cast<float*>(static_cast<unsigned char*>(ws) + P.off_partials);
    const int image_cols = P.col_groups * kPassCols;
    int pgrid = (image_cols * 32 * ng + 255) / 256;
    if (pgrid > sms * 4) pgrid = sms * 4;
    k_prepare_batched<<<pgrid, 256, 0, s>>>(xh, K, image_cols, batch, ng, xqb, counters, P.tile_groups);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(P.ctas));
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
    if (ng == 1)
        return cudaLaunchKernelEx(&cfg, k_gemv_batched<1>, tb, cd, row_scales, xh, tl, y, N, K, B, batch,
                                  static_cast<const uint32_t*>(xqb), counters, partials, P.tile_groups, P.col_groups);
    return cudaLaunchKernelEx(&cfg, k_gemv_batched<2>, tb, cd, row_scales, xh, tl, y, N, K, B, batch,
                              static_cast<const uint32_t*>(xqb), counters, partials, P.tile_groups, P.col_groups);
}

}  // namespace tetra
