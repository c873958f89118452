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
#include "tetra_device.cuh"

namespace tetra {
namespace {

constexpr int kQ4Threads = 512;
constexpr int kQ4Warps = kQ4Threads / 32;

// Packed layout (uint4 units): tile (strip, kt) at (strip * KT + kt) * 32 + lane, KT = K / 64; lane = 4 g + t
// owns four words m = 0..3; word m, nibbles n0..n7 (n_i at bits 4 i), weights of columns
// c = 64 kt + 16 t + 4 m + {0,1,2,3}:
//     n0, n4 = row g,     c + 0, c + 1        n1, n5 = row g,     c + 2, c + 3
//     n2, n6 = row g + 8, c + 0, c + 1        n3, n7 = row g + 8, c + 2, c + 3
// After the tiles: (scale, offset) half2 records at so_base + (strip * groups + group) * 16 + row.
__host__ __device__ inline size_t q4_weight_bytes(int strips, int K) { return size_t(strips) * (K / 64) * 512; }

__global__ void __launch_bounds__(256) k_q4_pack(const uint8_t* __restrict__ q, const __half* __restrict__ scale,
                                                 const __half* __restrict__ offset, uint32_t* __restrict__ packed,
                                                 int N, int K, int G) {
    const int strips = (N + 15) / 16, KT = K / 64, groups = K / G;
    const size_t words = size_t(strips) * KT * 128;
    const size_t so_words = size_t(strips) * groups * 16;
    uint32_t* so = packed + words;
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < words + so_words;
         i += size_t(gridDim.x) * blockDim.x) {
        if (i < words) {
            const int m = int(i & 3), lane = int((i >> 2) & 31);
            const size_t tile = i >> 7;
            const int kt = int(tile % KT), strip = int(tile / KT);
            const int g = lane >> 2, t = lane & 3;
            const int c = 64 * kt + 16 * t + 4 * m;  // multiple of 4: two whole bytes per row
            uint32_t w = 0;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int row = 16 * strip + g + 8 * half;
                if (row < N) {
                    const uint8_t* src = q + size_t(row) * (K / 2) + c / 2;
                    const uint32_t b0 = src[0], b1 = src[1];  // b0 = weights c, c+1; b1 = c+2, c+3
                    const uint32_t n_c0 = b0 & 15, n_c1 = b0 >> 4, n_c2 = b1 & 15, n_c3 = b1 >> 4;
                    // half 0: n0, n4, n1, n5; half 1: n2, n6, n3, n7
                    w |= (n_c0 << (8 * half)) | (n_c1 << (16 + 8 * half)) | (n_c2 << (4 + 8 * half)) |
                         (n_c3 << (20 + 8 * half));
                }
            }
            packed[i] = w;
        } else {
            const size_t j = i - words;
            const int r = int(j & 15);
            const size_t sg = j >> 4;
            const int group = int(sg % groups), strip = int(sg / groups);
            const int row = 16 * strip + r;
            uint32_t v = 0;
            if (row < N) {
                const size_t at = size_t(row) * groups + group;
                v = uint32_t(__half_as_ushort(scale[at])) | (uint32_t(__half_as_ushort(offset[at])) << 16);
            }
            so[j] = v;
        }
    }
}

__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t lop_and_or(uint32_t a, uint32_t mask, uint32_t magic) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(magic));  // (a & mask) | magic
    return r;
}

__device__ __forceinline__ void team_barrier(int team, int team_warps) {
    if (team_warps == 1)
        __syncwarp();
    else
        asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(team_warps * 32) : "memory");
}

// A team of S warps (S a power of two, 1..16) owns a strip of 16 rows at a time and splits its groups:
// warp p of the team takes groups p, p + S, ...  Per group: TPG = G / 64 tiles, four MMAs each, into one
// accumulator; then the bias correction, scale and offset.  At the end of a strip the team's warps add
// their sums through shared memory (two buffers, one named barrier per strip).
template <int G>
__global__ void __launch_bounds__(kQ4Threads, 2)
k_q4_gemv(const uint4* __restrict__ packed, const __half* __restrict__ x, float* __restrict__ y, int N, int K,
          int batch, int S) {
    constexpr int TPG = G / 64;
    extern __shared__ __align__(16) unsigned char q4_smem[];
    const int groups = K / G, KT = K / 64, strips = (N + 15) / 16;
    float2* gs = reinterpret_cast<float2*>(q4_smem);                                // [groups][8]: (sum x, sum bias x)
    float* red = reinterpret_cast<float*>(q4_smem + size_t(groups) * 64);           // [2][warps][128]
    const uint32_t* so = reinterpret_cast<const uint32_t*>(packed + size_t(strips) * KT * 32);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    pdl_release();
    pdl_wait();  // x may come from the preceding kernel

    // per (group, vector): sum of x and of bias_k x_k, bias 1024 for k % 4 in {0, 1}, 64 for {2, 3}
    for (int task = threadIdx.x; task < groups * 8; task += kQ4Threads) {
        const int v = task & 7, gi = task >> 3;
        float sx = 0.f, sb = 0.f;
        if (v < batch) {
            const uint2* src = reinterpret_cast<const uint2*>(x + size_t(v) * K + size_t(gi) * G);
            float lo = 0.f, hi = 0.f;  // k % 4 in {0, 1} / {2, 3}
            for (int i = 0; i < G / 4; ++i) {
                const uint2 u = __ldg(src + i);
                const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&u.x));
                const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
                lo += a.x + a.y;
                hi += b.x + b.y;
            }
            sx = lo + hi;
            sb = 1024.f * lo + 64.f * hi;
        }
        gs[task] = make_float2(sx, sb);
    }
    __syncthreads();

    const int teams = kQ4Warps / S, team = warp / S, p = warp % S;
    const __half* xv = x + size_t(g) * K + 16 * t;  // vector g (columns of B), this lane's 16 activations per tile
    const bool has_x = g < batch;
    int buf = 0;
    for (int strip = blockIdx.x * teams + team; strip < strips; strip += gridDim.x * teams) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const uint4* wrow = packed + size_t(strip) * KT * 32 + lane;
        const uint32_t* sorow = so + size_t(strip) * groups * 16 + g;
        // software pipeline over this warp's groups: the next group's weights are in flight during the MMAs
        uint4 wn[TPG];
        uint32_t so0n = 0, so1n = 0;
        if (p < groups) {
#pragma unroll
            for (int j = 0; j < TPG; ++j) wn[j] = __ldcs(wrow + size_t(p * TPG + j) * 32);
            so0n = __ldg(sorow + p * 16);
            so1n = __ldg(sorow + p * 16 + 8);
        }
        for (int gi = p; gi < groups; gi += S) {
            uint4 w[TPG];
#pragma unroll
            for (int j = 0; j < TPG; ++j) w[j] = wn[j];
            const uint32_t so0 = so0n, so1 = so1n;
            if (gi + S < groups) {
#pragma unroll
                for (int j = 0; j < TPG; ++j) wn[j] = __ldcs(wrow + size_t((gi + S) * TPG + j) * 32);
                so0n = __ldg(sorow + (gi + S) * 16);
                so1n = __ldg(sorow + (gi + S) * 16 + 8);
            }
            float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < TPG; ++j) {
                uint4 xa = make_uint4(0, 0, 0, 0), xb = make_uint4(0, 0, 0, 0);
                if (has_x) {
                    const uint4* xs = reinterpret_cast<const uint4*>(xv + size_t(gi * TPG + j) * 64);
                    xa = __ldg(xs);
                    xb = __ldg(xs + 1);
                }
                const uint32_t xr[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
                const uint32_t ww[4] = {w[j].x, w[j].y, w[j].z, w[j].w};
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const uint32_t w8 = ww[m] >> 8;
                    uint32_t a[4];
                    a[0] = lop_and_or(ww[m], 0x000F000Fu, 0x64006400u);  // row g,     columns c, c+1   (1024 + n)
                    a[1] = lop_and_or(w8, 0x000F000Fu, 0x64006400u);     // row g + 8, columns c, c+1
                    a[2] = lop_and_or(ww[m], 0x00F000F0u, 0x54005400u);  // row g,     columns c+2, c+3 (64 + n)
                    a[3] = lop_and_or(w8, 0x00F000F0u, 0x54005400u);     // row g + 8, columns c+2, c+3
                    mma_f16(d, a, xr[2 * m], xr[2 * m + 1]);
                }
            }
            // this lane's results: rows g (i = 0, 1) and g + 8 (i = 2, 3), vectors 2 t + (i & 1)
            const float4 cs = *reinterpret_cast<const float4*>(gs + gi * 8 + 2 * t);  // (sx, sb) of vectors 2t, 2t+1
            const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&so0));  // (scale, offset) of row g
            const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&so1));  // of row g + 8
            acc[0] += r0.x * (d[0] - cs.y) + r0.y * cs.x;
            acc[1] += r0.x * (d[1] - cs.w) + r0.y * cs.z;
            acc[2] += r1.x * (d[2] - cs.y) + r1.y * cs.x;
            acc[3] += r1.x * (d[3] - cs.w) + r1.y * cs.z;
        }
        // team sum in warp order, then store: element e = 4 lane + i is (row g + 8 (i / 2), vector 2 t + (i % 2))
        float* mine = red + (size_t(buf) * kQ4Warps + warp) * 128;
        *reinterpret_cast<float4*>(mine + 4 * lane) = make_float4(acc[0], acc[1], acc[2], acc[3]);
        team_barrier(team, S);
        const float* first = red + (size_t(buf) * kQ4Warps + team * S) * 128;
        for (int e = p * 32 + lane; e < 128; e += S * 32) {
            const int el = e >> 2, i = e & 3;
            const int row = 16 * strip + (el >> 2) + 8 * (i >> 1), v = 2 * (el & 3) + (i & 1);
            if (row < N && v < batch) {
                float total = 0.f;
                for (int k = 0; k < S; ++k) total += first[k * 128 + e];
                y[size_t(v) * N + row] = total;
            }
        }
        buf ^= 1;
    }
}

// One thread per (token, tile, t, m): four consecutive weights of the row as float16 (Sec. 4.4).
__global__ void __launch_bounds__(256) k_q4_rows(const uint32_t* __restrict__ packed, const int32_t* __restrict__ ids,
                                                 int count, __half* __restrict__ out, int N, int K, int G) {
    const int strips = (N + 15) / 16, KT = K / 64, groups = K / G;
    const uint32_t* so = packed + size_t(strips) * KT * 128;
    const size_t per_row = size_t(KT) * 16;
    pdl_release();
    pdl_wait();  // the ids may come from the preceding kernel
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < size_t(count) * per_row;
         i += size_t(gridDim.x) * blockDim.x) {
        const int tok = int(i / per_row);
        const int rem = int(i % per_row);
        const int m = rem & 3, t = (rem >> 2) & 3, kt = rem >> 4;
        const int c = 64 * kt + 16 * t + 4 * m;
        const int row = ids[tok];
        uint2 res = make_uint2(0u, 0u);
        if (row >= 0 && row < N) {
            const int strip = row >> 4, g = row & 7, half = (row >> 3) & 1;
            const uint32_t w = packed[((size_t(strip) * KT + kt) * 32 + g * 4 + t) * 4 + m] >> (8 * half);
            const uint32_t rec = so[(size_t(strip) * groups + c / G) * 16 + (row & 15)];
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

template <int G>
cudaError_t launch_q4_gemv(const void* packed, const void* x, float* y, int N, int K, int batch, int sms,
                           cudaStream_t s) {
    const int strips = (N + 15) / 16, groups = K / G;
    // team size: enough (strip, group-slice) units for two CTAs of 16 warps per SM
    int S = 1;
    while (S < kQ4Warps && S * 2 <= groups && size_t(strips) * S < size_t(2) * sms * kQ4Warps) S *= 2;
    const int teams = kQ4Warps / S;
    int grid = (strips + teams - 1) / teams;
    if (grid > 2 * sms) grid = 2 * sms;
    const size_t smem = size_t(groups) * 64 + size_t(2) * kQ4Warps * 128 * 4;
    static bool attr_set[2] = {false, false};
    if (!attr_set[G == 128]) {
        cudaError_t e = cudaFuncSetAttribute(k_q4_gemv<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[G == 128] = true;
    }
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
    return cudaLaunchKernelEx(&cfg, k_q4_gemv<G>, static_cast<const uint4*>(packed), static_cast<const __half*>(x), y,
                              N, K, batch, S);
}

}  // namespace
}  // namespace tetra

using namespace tetra;

extern "C" {

size_t tetra_q4_packed_bytes(int N, int K, int G) {
    if (check_shape(N, K, G) != TETRA_OK) return 0;
    const int strips = (N + 15) / 16;
    return q4_weight_bytes(strips, K) + size_t(strips) * (K / G) * 16 * 4;
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
    if (size_t(K / G) * 64 + 16384 > 96 * 1024) return TETRA_ERR_SHAPE;
    int sms = 0;
    const int drc = device_sm_count(&sms);
    if (drc != TETRA_OK) return drc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return cuda_status(G == 128 ? launch_q4_gemv<128>(packed_dev, x_dev, y_dev, N, K, batch, sms, s)
                                : launch_q4_gemv<64>(packed_dev, x_dev, y_dev, N, K, batch, sms, s));
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
    return cuda_status(cudaLaunchKernelEx(&cfg, k_q4_rows, static_cast<const uint32_t*>(packed_dev), ids_dev, count,
                                          static_cast<__half*>(out_dev), N, K, G));
}

}  // extern "C"
