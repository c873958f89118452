// Decode-only kernels and the HBM code layout (pack) kernel.
#include "tetra_device.cuh"
#include "tetra_launch.h"

namespace tetra {

// ---------------------------------------------------------------------------
// tetra_decode_blocks: file-order words -> 24 coordinates (+ m, g).  One thread
// per block; the paper-format tables are read through the read-only cache.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_decode_file(const uint8_t* __restrict__ codes,
                                                     const DeviceTables* __restrict__ tab,
                                                     int8_t* __restrict__ y_out, uint8_t* __restrict__ mg_out,
                                                     size_t nblocks) {
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < nblocks;
         i += size_t(gridDim.x) * blockDim.x) {
        int y[24], m, g;
        decode_file_word(&tab->paper, load_file_word(codes, i), y, &m, &g);
        uint32_t* dst = reinterpret_cast<uint32_t*>(y_out + 24 * i);  // 24 i is a multiple of 4
#pragma unroll
        for (int k = 0; k < 6; ++k)
            dst[k] = uint32_t(y[4 * k] & 0xFF) | (uint32_t(y[4 * k + 1] & 0xFF) << 8) |
                     (uint32_t(y[4 * k + 2] & 0xFF) << 16) | (uint32_t(y[4 * k + 3] & 0xFF) << 24);
        if (mg_out) {
            mg_out[2 * i] = uint8_t(m);
            mg_out[2 * i + 1] = uint8_t(g);
        }
    }
}

// ---------------------------------------------------------------------------
// Packed layout.  Rows are taken in groups of eight; for row group G and block
// column c the eight words form a 48-byte record split into three 16-byte
// parts, stored as  packed[(G * 3 + part) * B + c]  (uint4 units):
//   part 0: w0 of rows 8G+0..3      part 1: w0 of rows 8G+4..7
//   part 2: w1 of rows 8G+0..7 (two per 32-bit lane, even row in the low half)
// so a warp whose lanes own consecutive columns reads 512 contiguous bytes per
// part.  Rows beyond N are the all-zero word (the origin).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_pack(const uint8_t* __restrict__ codes,
                                              const DeviceTables* __restrict__ tab,
                                              uint4* __restrict__ packed, int N, int B) {
    const int groups = (N + 7) / 8;
    const size_t total = size_t(groups) * B;
    for (size_t t = blockIdx.x * size_t(blockDim.x) + threadIdx.x; t < total;
         t += size_t(gridDim.x) * blockDim.x) {
        const int G = int(t / B), c = int(t % B);
        uint32_t w0[8], w1[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int row = 8 * G + r;
            const uint64_t w = row < N ? load_file_word(codes, size_t(row) * B + c) : 0ull;
            file_to_device_word(w, tab, &w0[r], &w1[r]);
        }
        uint4* rec = packed + size_t(G) * 3 * B + c;
        rec[0] = make_uint4(w0[0], w0[1], w0[2], w0[3]);
        rec[B] = make_uint4(w0[4], w0[5], w0[6], w0[7]);
        rec[2 * size_t(B)] = make_uint4(w1[0] | (w1[1] << 16), w1[2] | (w1[3] << 16),
                                        w1[4] | (w1[5] << 16), w1[6] | (w1[7] << 16));
    }
}

// ---------------------------------------------------------------------------
// tetra_decode_packed: the GEMV's own decoder, emitting coordinates instead of
// multiplying.  One thread per (row group, column) record.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void emit_block(const FastBlock& fb, int8_t* __restrict__ y_out,
                                           uint8_t* __restrict__ mg_out, size_t block) {
    int y[24];
#pragma unroll
    for (int k = 0; k < 6; ++k)
#pragma unroll
        for (int i = 0; i < 4; ++i) y[4 * k + i] = -int(int8_t((fb.y[k] >> (8 * i)) & 0xFF));  // the decoder emits -y
    int norm = 0;
#pragma unroll
    for (int k = 0; k < 24; ++k) norm += y[k] * y[k];
    uint32_t* dst = reinterpret_cast<uint32_t*>(y_out + 24 * block);
#pragma unroll
    for (int k = 0; k < 6; ++k)
        dst[k] = uint32_t(y[4 * k] & 0xFF) | (uint32_t(y[4 * k + 1] & 0xFF) << 8) |
                 (uint32_t(y[4 * k + 2] & 0xFF) << 16) | (uint32_t(y[4 * k + 3] & 0xFF) << 24);
    if (mg_out) {
        mg_out[2 * block] = uint8_t(norm >> 4);
        mg_out[2 * block + 1] = uint8_t((fb.goff >> 3) & 1u);
    }
}

__global__ void __launch_bounds__(256) k_decode_packed(const uint4* __restrict__ packed,
                                                       const DeviceTables* __restrict__ tab,
                                                       int8_t* __restrict__ y_out, uint8_t* __restrict__ mg_out,
                                                       int N, int B) {
    extern __shared__ __align__(16) unsigned char smem[];
    const uint32_t sm_tab = smem_u32(stage_fast_tables(tab, smem));
    __syncthreads();
    const int groups = (N + 7) / 8;
    const size_t total = size_t(groups) * B;
    for (size_t t = blockIdx.x * size_t(blockDim.x) + threadIdx.x; t < total;
         t += size_t(gridDim.x) * blockDim.x) {
        const int G = int(t / B), c = int(t % B);
        const uint4* rec = packed + size_t(G) * 3 * B + c;
        const uint4 lo = rec[0], hi = rec[B], w1 = rec[2 * size_t(B)];
        const uint32_t w0[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
        const uint32_t w1p[4] = {w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int row = 8 * G + r;
            if (row >= N) break;
            FastBlock fb;
            if (r & 1) fast_decode<true>(sm_tab, w0[r], w1p[r >> 1], fb);
            else fast_decode<false>(sm_tab, w0[r], w1p[r >> 1], fb);
            emit_block(fb, y_out, mg_out, size_t(row) * B + c);
        }
    }
}

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------
static int grid_for(size_t items, int threads, int cap) {
    size_t g = (items + threads - 1) / threads;
    if (g > size_t(cap)) g = size_t(cap);
    if (g == 0) g = 1;
    return int(g);
}

cudaError_t launch_decode_file(const void* codes, const void* table, int8_t* y, uint8_t* mg, size_t nblocks,
                               cudaStream_t s) {
    k_decode_file<<<grid_for(nblocks, 256, 148 * 32), 256, 0, s>>>(
        static_cast<const uint8_t*>(codes), static_cast<const DeviceTables*>(table), y, mg, nblocks);
    return cudaGetLastError();
}

cudaError_t launch_pack(const void* codes, const void* table, void* packed, int N, int B, cudaStream_t s) {
    const size_t items = size_t((N + 7) / 8) * B;
    k_pack<<<grid_for(items, 256, 148 * 32), 256, 0, s>>>(static_cast<const uint8_t*>(codes),
                                                            static_cast<const DeviceTables*>(table),
                                                            static_cast<uint4*>(packed), N, B);
    return cudaGetLastError();
}

cudaError_t launch_decode_packed(const void* packed, const void* table, int8_t* y, uint8_t* mg, int N, int B,
                                 cudaStream_t s) {
    const size_t items = size_t((N + 7) / 8) * B;
    k_decode_packed<<<grid_for(items, 256, 148 * 4), 256, kTableSmemBytes, s>>>(
        static_cast<const uint4*>(packed), static_cast<const DeviceTables*>(table), y, mg, N, B);
    return cudaGetLastError();
}

}  // namespace tetra
