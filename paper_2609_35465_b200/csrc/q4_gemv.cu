// 4-bit group-quantised matrices: device layout, matrix-vector product, row dequantisation
// (Sec. 4.1 and 4.3: int4 records, groups of 128; Sec. 4.4: embedding table and output head, groups of
// 64; Sec. 5.1: dequantise with the group's scale and offset, accumulate in float32).
//
// The product is bound by HBM (4.25 or 4.5 bits per weight), so the kernel is built around bytes in
// flight and instructions per byte.  A 32-bit word of eight nibbles becomes four float16x2 operand
// registers with five logic operations:  (w & 0x000F000F) | 0x64006400 is the pair (1024 + n0, 1024 + n4),
// (w & 0x00F000F0) | 0x54005400 is (64 + n1, 64 + n5), and the same two masks on w >> 8 give n2, n6 and n3,
// n7.  The packed layout puts the nibbles where mma.sync.m16n8k16 wants them, so those registers ARE the A
// fragment of a 16-row x 16-weight tile; the activations are the B fragment (column v = vector v, so up to
// eight vectors cost the same as one), products of exact float16 values are accumulated in float32 inside
// the MMA, one accumulator per group; the biases 1024 and 64 are removed with the group's precomputed
// sum(bias_k x_k), then scale and offset are applied in float32:
//     y += scale * (D - C_group) + offset * sum_group(x).
// Tensor cores are used here as the cheapest exact multiply-accumulate (six instructions per 256 weights),
// not because the product is compute-bound: at one FFMA per weight the FP32 pipes would be the limit.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/tetra.h"
#include "../../include/tetra_q4.h"
#include "q4_common.cuh"
#include "tetra_device.cuh"
#include "tetra_launch.h"

namespace tetra {
namespace {

#ifndef TETRA_Q4_THREADS
#define TETRA_Q4_THREADS 512
#define TETRA_Q4_CTAS 1
#endif
constexpr int kQ4Threads = TETRA_Q4_THREADS;
constexpr int kQ4CtasPerSm = TETRA_Q4_CTAS;
constexpr int kQ4Warps = kQ4Threads / 32;

__global__ void __launch_bounds__(256) k_q4_pack(const uint8_t* __restrict__ q, const __half* __restrict__ scale,
                                                 const __half* __restrict__ offset, uint32_t* __restrict__ packed,
                                                 int N, int K, int G) {
    const int strips = (N + 31) / 32, groups = K / G, chunk_words = q4_chunk_bytes(G) / 4, tile_words = (G / 64) * 256;
    const size_t total = size_t(strips) * groups * chunk_words;
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < total; i += size_t(gridDim.x) * blockDim.x) {
        const int wi = int(i % chunk_words);
        const size_t sg = i / chunk_words;
        const int group = int(sg % groups), strip = int(sg / groups);
        uint32_t w = 0;
        if (wi < tile_words) {
            const int m = wi & 3, lane = (wi >> 2) & 31, h = (wi >> 7) & 1, j = wi >> 8;
            const int g = lane >> 2, t = lane & 3;
            const int c = group * G + 64 * j + 16 * t + 4 * m;  // multiple of 4: two whole bytes per row
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int row = 32 * strip + 16 * h + g + 8 * half;
                if (row < N) {
                    const uint8_t* src = q + size_t(row) * (K / 2) + c / 2;
                    const uint32_t b0 = src[0], b1 = src[1];  // b0 = weights c, c+1; b1 = c+2, c+3
                    const uint32_t n_c0 = b0 & 15, n_c1 = b0 >> 4, n_c2 = b1 & 15, n_c3 = b1 >> 4;
                    // half 0: n0, n4, n1, n5; half 1: n2, n6, n3, n7
                    w |= (n_c0 << (8 * half)) | (n_c1 << (16 + 8 * half)) | (n_c2 << (4 + 8 * half)) |
                         (n_c3 << (20 + 8 * half));
                }
            }
        } else {
            const int row = 32 * strip + (wi - tile_words);
            if (row < N) {
                const size_t at = size_t(row) * groups + group;
                w = uint32_t(__half_as_ushort(scale[at])) | (uint32_t(__half_as_ushort(offset[at])) << 16);
            }
        }
        packed[i] = w;
    }
}

// A CTA owns a contiguous range of 32-row strips (equal shares), and its 16 warps cut the CTA's chunks, in
// memory order, into 16 equal contiguous ranges: every warp streams one contiguous piece of the matrix
// through a ring of DEPTH slots in shared memory (cp.async, DEPTH - 1 chunks ahead).  Per chunk: the
// accumulators of the two 16-row sub-tiles start at minus the group's sum(bias_k x_k), every 64-column tile
// adds four MMAs per sub-tile (the activations' B fragments are shared by both), then
//     acc += scale * D + offset * sum_group(x).
// A strip that lies wholly inside a warp's range is stored directly; a strip cut by a range boundary leaves
// one piece per warp in shared memory, and after one CTA barrier the pieces are added in warp order.
// Addresses advance by running pointers: the loop body is dequantise, multiply, scale.
// XS: the activations are staged in shared memory (rows padded by 16 bytes so that the eight vectors' reads
// fall into different banks); otherwise they are read through L1.
template <int G, int DEPTH, bool XS>
__global__ void __launch_bounds__(kQ4Threads, kQ4CtasPerSm)
k_q4_gemv(const unsigned char* __restrict__ packed, const __half* __restrict__ x, float* __restrict__ y, int N, int K,
          int batch) {
    constexpr int TPG = G / 64, CH = q4_chunk_bytes(G), PIECES = CH / 16;
    extern __shared__ __align__(16) unsigned char q4_smem[];
    __shared__ int piece_strip[2 * kQ4Warps];
    const int groups = K / G, strips = (N + 31) / 32;
    float2* gs = reinterpret_cast<float2*>(q4_smem);                        // [groups][8]: (sum x, -sum bias x)
    float* pieces = reinterpret_cast<float*>(q4_smem + size_t(groups) * 64);  // [warps][2][256]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kPieceBytes = kQ4Warps * 2 * 1024;
    const uint32_t ring = smem_u32(q4_smem + size_t(groups) * 64 + kPieceBytes) + uint32_t(warp) * (DEPTH * CH);
    unsigned char* xs_base = q4_smem + size_t(groups) * 64 + kPieceBytes + size_t(kQ4Warps) * DEPTH * CH;
    const uint32_t xs_stride = uint32_t(K) * 2u + 16u;  // bytes per staged vector
    const int g = lane >> 2, t = lane & 3;
    pdl_release();
    if (threadIdx.x < 2 * kQ4Warps) piece_strip[threadIdx.x] = -1;

    // this CTA's strips, this warp's chunks (local index n = local strip * groups + group)
    const int strip_begin = int(size_t(blockIdx.x) * strips / gridDim.x);
    const int strip_end = int((size_t(blockIdx.x) + 1) * strips / gridDim.x);
    const uint32_t cta_chunks = uint32_t(strip_end - strip_begin) * uint32_t(groups);
    const uint32_t n_begin = uint32_t(uint64_t(warp) * cta_chunks / kQ4Warps);
    const uint32_t n_end = uint32_t((uint64_t(warp) + 1) * cta_chunks / kQ4Warps);
    // running addresses: f_src = next chunk to copy (this lane's 16 bytes of each 512), f_todo = chunks left to
    // copy; slot_lane = this lane's 16 bytes in the slot being consumed; the slot consumed last is refilled
    const unsigned char* f_src = packed + (size_t(strip_begin) * groups + n_begin) * CH + lane * 16;
    int f_todo = int(n_end - n_begin);
    const uint32_t ring_lane = ring + lane * 16, ring_lane_end = ring_lane + DEPTH * CH;
    const bool tail_lane = lane < PIECES % 32;  // lanes that copy the last, partial group of 16-byte pieces
    auto fetch_into = [&](uint32_t dst_lane) {
        if (f_todo > 0) {
#pragma unroll
            for (int i = 0; i < PIECES / 32; ++i) q4_cp_async16(dst_lane + i * 512, f_src + i * 512);
            if (PIECES % 32 != 0 && tail_lane) q4_cp_async16(dst_lane + (PIECES / 32) * 512, f_src + (PIECES / 32) * 512);
            f_src += CH;
        }
        --f_todo;
        asm volatile("cp.async.commit_group;" ::: "memory");  // one group per call, empty or not
    };
#pragma unroll
    for (int i = 0; i < DEPTH - 1; ++i) fetch_into(ring_lane + i * CH);  // the weights do not depend on the preceding kernel

    pdl_wait();  // x may come from the preceding kernel
    if (XS) {
        for (int i = threadIdx.x; i < batch * (K / 8); i += kQ4Threads) {
            const int v = i / (K / 8), c8 = i % (K / 8);
            *reinterpret_cast<uint4*>(xs_base + size_t(v) * xs_stride + size_t(c8) * 16) =
                __ldg(reinterpret_cast<const uint4*>(x + size_t(v) * K) + c8);
        }
        __syncthreads();
    }
    // per (group, vector): sum of x and minus the sum of bias_k x_k, bias 1024 for k % 4 in {0, 1}, 64 for {2, 3};
    // eight lanes per task, combined by shuffles in a fixed order
    for (int task0 = (threadIdx.x >> 3); task0 < groups * 8; task0 += kQ4Threads / 8) {
        const int v = task0 & 7, gi = task0 >> 3, sub = threadIdx.x & 7;
        float lo = 0.f, hi = 0.f;  // k % 4 in {0, 1} / {2, 3}
        if (v < batch) {
            const uint2* src = XS ? reinterpret_cast<const uint2*>(xs_base + size_t(v) * xs_stride) + size_t(gi) * (G / 4)
                                  : reinterpret_cast<const uint2*>(x + size_t(v) * K + size_t(gi) * G);
#pragma unroll
            for (int i = 0; i < G / 32; ++i) {
                const uint2 u = XS ? src[sub + 8 * i] : __ldg(src + sub + 8 * i);
                const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&u.x));
                const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
                lo += a.x + a.y;
                hi += b.x + b.y;
            }
        }
#pragma unroll
        for (int o = 4; o >= 1; o >>= 1) {
            lo += __shfl_xor_sync(0xFFFFFFFFu, lo, o);
            hi += __shfl_xor_sync(0xFFFFFFFFu, hi, o);
        }
        if (sub == 0) gs[task0] = make_float2(lo + hi, -(1024.f * lo + 64.f * hi));
    }
    __syncthreads();

    // column g of B is vector g; columns at or beyond batch are never stored, so they may hold any vector
    const uint32_t x_vec = uint32_t(g < batch ? g : batch - 1);
    // this lane's 16 activations of the first tile of group 0: an offset in halves (global) or a shared address
    const uint32_t x_lane = XS ? smem_u32(xs_base) + x_vec * xs_stride + 32u * t : x_vec * uint32_t(K) + 16u * t;
    const uint32_t gs_lane = smem_u32(gs) + uint32_t(t) * 16;
    uint32_t slot_lane = ring_lane;                       // slot being consumed
    uint32_t refill_lane = ring_lane + (DEPTH - 1) * CH;  // slot consumed last (empty at the start)
    const uint32_t so_delta = uint32_t(TPG * 1024 + g * 4) - uint32_t(lane * 16);  // slot_lane -> this lane's scale records
    int gi = int(n_begin % uint32_t(groups));
    int strip = strip_begin + int(n_begin / uint32_t(groups));
    int n_pieces = 0;
    uint32_t left = n_end - n_begin;
    while (left > 0) {
        // one segment: the chunks of this warp that belong to one strip
        const int seg_first = gi;
        const uint32_t seg_len = min(uint32_t(groups - gi), left);
        uint32_t xo = x_lane + uint32_t(gi) * G * (XS ? 2u : 1u);
        uint32_t gsp = gs_lane + uint32_t(gi) * 64;
        float acc[2][4];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[h][i] = 0.f;
        for (uint32_t c = 0; c < seg_len; ++c) {
            uint32_t cs[4];  // (sum x, -sum bias x) of vectors 2 t, 2 t + 1
            q4_lds128(gsp, cs);
            fetch_into(refill_lane);
            q4_cp_async_wait<DEPTH - 1>();  // this chunk has landed
            __syncwarp();
            float d[2][4];
#pragma unroll
            for (int j = 0; j < TPG; ++j) {
                uint32_t xr[8];
                if (XS) {
                    uint32_t lo[4], hi[4];
                    q4_lds128(xo + 128 * j, lo);
                    q4_lds128(xo + 128 * j + 16, hi);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        xr[i] = lo[i];
                        xr[4 + i] = hi[i];
                    }
                } else {
                    const uint4* xg = reinterpret_cast<const uint4*>(x + xo) + 8 * j;  // L1-resident activations
                    const uint4 xa = __ldg(xg);
                    const uint4 xb = __ldg(xg + 1);
                    xr[0] = xa.x; xr[1] = xa.y; xr[2] = xa.z; xr[3] = xa.w;
                    xr[4] = xb.x; xr[5] = xb.y; xr[6] = xb.z; xr[7] = xb.w;
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t ww[4];
                    q4_lds128(slot_lane + j * 1024 + h * 512, ww);
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        uint32_t a[4];
                        const uint32_t w8 = ww[m] >> 8;
                        a[0] = lop_and_or(ww[m], 0x000F000Fu, 0x64006400u);  // row g,     columns c, c+1   (1024 + n)
                        a[1] = lop_and_or(w8, 0x000F000Fu, 0x64006400u);     // row g + 8, columns c, c+1
                        a[2] = lop_and_or(ww[m], 0x00F000F0u, 0x54005400u);  // row g,     columns c+2, c+3 (64 + n)
                        a[3] = lop_and_or(w8, 0x00F000F0u, 0x54005400u);     // row g + 8, columns c+2, c+3
                        if (j == 0 && m == 0)
                            mma_f16_first(d[h], a, xr[0], xr[1], __uint_as_float(cs[1]), __uint_as_float(cs[3]));
                        else
                            mma_f16(d[h], a, xr[2 * m], xr[2 * m + 1]);
                    }
                }
            }
            // this lane's results: rows 16 h + g (i = 0, 1) and 16 h + g + 8 (i = 2, 3), vectors 2 t + (i & 1)
            const float sx_even = __uint_as_float(cs[0]), sx_odd = __uint_as_float(cs[2]);
            const uint32_t so_lane = slot_lane + so_delta;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint32_t so0 = lds32(so_lane + 64 * h);
                const uint32_t so1 = lds32(so_lane + 64 * h + 32);
                const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&so0));  // (scale, offset)
                const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&so1));
                fma2(r0.y, sx_even, sx_odd, acc[h][0], acc[h][1]);  // offset * sum(x), vectors 2 t and 2 t + 1
                fma2(r0.x, d[h][0], d[h][1], acc[h][0], acc[h][1]);  // scale * (sum q x)
                fma2(r1.y, sx_even, sx_odd, acc[h][2], acc[h][3]);
                fma2(r1.x, d[h][2], d[h][3], acc[h][2], acc[h][3]);
            }
            __syncwarp();  // every lane has read the slot before the next refill targets it
            refill_lane = slot_lane;
            slot_lane += CH;
            if (slot_lane == ring_lane_end) slot_lane = ring_lane;
            xo += G * (XS ? 2u : 1u);
            gsp += 64;
        }
        left -= seg_len;
        gi += int(seg_len);
        // element e = 8 lane + 4 h + i is (row 16 h + g + 8 (i / 2), vector 2 t + (i % 2)) of the strip
        if (seg_first == 0 && gi == groups) {  // the whole strip was this warp's
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = 32 * strip + 16 * h + g + 8 * (i >> 1), v = 2 * t + (i & 1);
                    if (row < N && v < batch) y[size_t(v) * N + row] = acc[h][i];
                }
        } else {  // a strip shared with a neighbouring warp: leave a piece
            float* mine = pieces + (2 * warp + n_pieces) * 256 + 8 * lane;
            *reinterpret_cast<float4*>(mine) = make_float4(acc[0][0], acc[0][1], acc[0][2], acc[0][3]);
            *reinterpret_cast<float4*>(mine + 4) = make_float4(acc[1][0], acc[1][1], acc[1][2], acc[1][3]);
            if (lane == 0) piece_strip[2 * warp + n_pieces] = strip;
            ++n_pieces;
        }
        if (gi == groups) {
            gi = 0;
            ++strip;
        }
    }
    q4_cp_async_wait<0>();
    __syncthreads();
    // pieces in (warp, first/second) order are in memory order: the pieces of a strip are consecutive
    if (threadIdx.x < 256) {
        const int e = threadIdx.x, el = e >> 3, h = (e >> 2) & 1, i = e & 3;
        const int r_in = 16 * h + (el >> 2) + 8 * (i >> 1), v = 2 * (el & 3) + (i & 1);
        int cur = -1;
        float total = 0.f;
        for (int pc = 0; pc <= 2 * kQ4Warps; ++pc) {
            const int sidx = pc < 2 * kQ4Warps ? piece_strip[pc] : -2;
            if (sidx == -1) continue;
            if (sidx != cur) {
                if (cur >= 0 && 32 * cur + r_in < N && v < batch) y[size_t(v) * N + 32 * cur + r_in] = total;
                cur = sidx;
                total = 0.f;
            }
            if (sidx >= 0) total += pieces[pc * 256 + e];
        }
    }
}

// One thread per (token, four consecutive columns): float16 weights of the row (Sec. 4.4).
__global__ void __launch_bounds__(256) k_q4_rows(const unsigned char* __restrict__ packed, const int32_t* __restrict__ ids,
                                                 int count, __half* __restrict__ out, int N, int K, int G) {
    const int groups = K / G, CH = q4_chunk_bytes(G), tile_bytes = (G / 64) * 1024;
    const size_t per_row = size_t(K / 4);
    pdl_release();
    pdl_wait();  // the ids may come from the preceding kernel
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < size_t(count) * per_row;
         i += size_t(gridDim.x) * blockDim.x) {
        const int tok = int(i / per_row);
        const int c = 4 * int(i % per_row);
        const int row = ids[tok];
        uint2 res = make_uint2(0u, 0u);
        if (row >= 0 && row < N) {
            const int strip = row >> 5, rr = row & 31, h = rr >> 4, g = rr & 7, half = (rr >> 3) & 1;
            const int group = c / G, cg = c % G, j = cg >> 6, t = (cg >> 4) & 3, m = (cg >> 2) & 3;
            const unsigned char* chunk = packed + (size_t(strip) * groups + group) * CH;
            const uint32_t w = *reinterpret_cast<const uint32_t*>(chunk + j * 1024 + h * 512 + (g * 4 + t) * 16 + m * 4) >>
                               (8 * half);
            const uint32_t rec = *reinterpret_cast<const uint32_t*>(chunk + tile_bytes + rr * 4);
            const float2 sc = __half22float2(*reinterpret_cast<const __half2*>(&rec));
            const float n0 = float(w & 15u), n1 = float((w >> 16) & 15u);        // columns c, c + 1
            const float n2 = float((w >> 4) & 15u), n3 = float((w >> 20) & 15u);  // columns c + 2, c + 3
            const __half2 lo = __floats2half2_rn(__fmaf_rn(sc.x, n0, sc.y), __fmaf_rn(sc.x, n1, sc.y));
            const __half2 hi = __floats2half2_rn(__fmaf_rn(sc.x, n2, sc.y), __fmaf_rn(sc.x, n3, sc.y));
            res = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
        }
        *reinterpret_cast<uint2*>(out + size_t(tok) * K + c) = res;
    }
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? TETRA_OK : TETRA_ERR_CUDA; }

int check_shape(int N, int K, int G) {
    if (N <= 0 || K <= 0 || K > TETRA_Q4_MAX_K) return TETRA_ERR_SHAPE;
    if ((G != 64 && G != 128) || K % G) return TETRA_ERR_SHAPE;
    return TETRA_OK;
}

int device_sm_count(int* sms) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
    return cuda_status(e);
}

constexpr size_t kQ4SmemLimit = 224 * 1024 / kQ4CtasPerSm - 2048;
constexpr size_t kQ4StageLimit = 40 * 1024;  // activations up to this size are staged in shared memory

template <int G, int DEPTH, bool XS>
cudaError_t launch_q4_variant(const void* packed, const void* x, float* y, int N, int K, int batch, int sms,
                              cudaStream_t s) {
    const int strips = (N + 31) / 32, groups = K / G;
    int grid = strips < kQ4CtasPerSm * sms ? strips : kQ4CtasPerSm * sms;
    const size_t smem = size_t(groups) * 64 + size_t(kQ4Warps) * 2048 + size_t(kQ4Warps) * DEPTH * q4_chunk_bytes(G) +
                        (XS ? size_t(batch) * (size_t(K) * 2 + 16) : 0);
    static PerDeviceOnce once;  // per instantiation
    cudaError_t e = once.run([] {
        return cudaFuncSetAttribute(k_q4_gemv<G, DEPTH, XS>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kQ4SmemLimit));
    });
    if (e != cudaSuccess) return e;
    if (smem > kQ4SmemLimit) return cudaErrorInvalidValue;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid));
    cfg.blockDim = dim3(kQ4Threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_q4_gemv<G, DEPTH, XS>, static_cast<const unsigned char*>(packed),
                              static_cast<const __half*>(x), y, N, K, batch);
}

template <int G, int DEPTH>
cudaError_t launch_q4_gemv(const void* packed, const void* x, float* y, int N, int K, int batch, int sms,
                           cudaStream_t s) {
    if (size_t(batch) * (size_t(K) * 2 + 16) <= kQ4StageLimit)
        return launch_q4_variant<G, DEPTH, true>(packed, x, y, N, K, batch, sms, s);
    return launch_q4_variant<G, DEPTH, false>(packed, x, y, N, K, batch, sms, s);
}

}  // namespace
}  // namespace tetra

using namespace tetra;

extern "C" {

size_t tetra_q4_packed_bytes(int N, int K, int G) {
    if (check_shape(N, K, G) != TETRA_OK) return 0;
    return size_t((N + 31) / 32) * (K / G) * q4_chunk_bytes(G);
}

int tetra_q4_pack(const void* q_dev, const void* scale_dev, const void* offset_dev, void* packed_dev,
                  size_t packed_bytes, int N, int K, int G, void* stream) {
    if (!q_dev || !scale_dev || !offset_dev || !packed_dev) return TETRA_ERR_NULL;
    const int rc = check_shape(N, K, G);
    if (rc != TETRA_OK) return rc;
    if (!aligned(q_dev, 16) || !aligned(scale_dev, 16) || !aligned(offset_dev, 16) || !aligned(packed_dev, 16))
        return TETRA_ERR_ALIGN;
    const size_t need = tetra_q4_packed_bytes(N, K, G);
    if (packed_bytes < need) return TETRA_ERR_SIZE;
    const size_t items = need / 4;
    size_t grid = (items + 255) / 256;
    if (grid > 148 * 32) grid = 148 * 32;
    k_q4_pack<<<unsigned(grid), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint8_t*>(q_dev), static_cast<const __half*>(scale_dev),
        static_cast<const __half*>(offset_dev), static_cast<uint32_t*>(packed_dev), N, K, G);
    return cuda_status(cudaGetLastError());
}

int tetra_q4_gemv(const void* packed_dev, const void* x_dev, float* y_dev, int N, int K, int G, int batch,
                  void* stream) {
    if (!packed_dev || !x_dev || !y_dev) return TETRA_ERR_NULL;
    const int rc = check_shape(N, K, G);
    if (rc != TETRA_OK) return rc;
    if (batch < 1 || batch > TETRA_Q4_MAX_BATCH) return TETRA_ERR_BATCH;
    if (!aligned(packed_dev, 16) || !aligned(x_dev, 16) || !aligned(y_dev, 4)) return TETRA_ERR_ALIGN;
    int sms = 0;
    const int drc = device_sm_count(&sms);
    if (drc != TETRA_OK) return drc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return cuda_status(G == 128 ? launch_q4_gemv<128, 3>(packed_dev, x_dev, y_dev, N, K, batch, sms, s)
                                : launch_q4_gemv<64, 6>(packed_dev, x_dev, y_dev, N, K, batch, sms, s));
}

int tetra_q4_rows(const void* packed_dev, const int32_t* ids_dev, int count, void* out_dev, int N, int K, int G,
                  void* stream) {
    if (count == 0) return TETRA_OK;
    if (!packed_dev || !ids_dev || !out_dev) return TETRA_ERR_NULL;
    const int rc = check_shape(N, K, G);
    if (rc != TETRA_OK) return rc;
    if (count < 0) return TETRA_ERR_SHAPE;
    if (!aligned(packed_dev, 16) || !aligned(ids_dev, 4) || !aligned(out_dev, 8)) return TETRA_ERR_ALIGN;
    const size_t items = size_t(count) * (K / 4);
    size_t grid = (items + 255) / 256;
    if (grid > 148 * 16) grid = 148 * 16;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid));
    cfg.blockDim = dim3(256);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cuda_status(cudaLaunchKernelEx(&cfg, k_q4_rows, static_cast<const unsigned char*>(packed_dev), ids_dev, count,
                                          static_cast<__half*>(out_dev), N, K, G));
}

}  // extern "C"
