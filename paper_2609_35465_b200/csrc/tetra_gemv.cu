// Decode-and-multiply kernels (Eq. (2), Sec. 5.1) for sm_100a.
//
//   k_gemv_paper  the thread layout the paper describes for its own GPU: a warp
//                 per output row, a lane per block, the six table loads of
//                 Fig. "decode", FP32 multiply-accumulate, shuffle reduction.
//                 Kept as a comparison arm and cross-check.
//   k_gemv_fast   the B200 design: a lane owns one block column and keeps its
//                 24 activations in registers as 24-bit fixed point (three int8
//                 planes, power-of-two step per block column, so float16 inputs
//                 within 2^12 of the column's largest are held exactly); it
//                 walks the rows, decodes each word into packed int8 with PRMT
//                 lookups and multiplies with DP4A: products and the sum over
//                 a block are exact integers, one rounding when the block's sum
//                 becomes a float, FP32 accumulation across blocks.  The ALU
//                 pipe only unpacks fields; the integer-MAD pipe does the
//                 arithmetic.  One persistent grid serves one matrix or a list.
#include <cuda_fp16.h>

#include "tetra_device.cuh"
#include "tetra_launch.h"

namespace tetra {

// ===========================================================================
// Paper-design kernel
// ===========================================================================
constexpr int kPaperTile = 64;  // blocks of x per shared-memory tile (the paper's T)

__global__ void __launch_bounds__(256) k_gemv_paper(const uint8_t* __restrict__ codes, size_t row_stride,
                                                    const float* __restrict__ row_scales,
                                                    const DeviceTables* __restrict__ tab,
                                                    const __half* __restrict__ x, float* __restrict__ y, int N, int K,
                                                    int B, int ntail, const __half* __restrict__ tail) {
    __shared__ PaperTables T;
    __shared__ float gain[2];
    __shared__ float xt[kPaperTile * 24];
    {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(&tab->paper);
        uint32_t* dst = reinterpret_cast<uint32_t*>(&T);
        for (int i = threadIdx.x; i < int(sizeof(PaperTables) / 4); i += blockDim.x) dst[i] = src[i];
        if (threadIdx.x < 2) gain[threadIdx.x] = tab->gain[threadIdx.x];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = blockIdx.x * 8 + warp;
    const __half* xb = x + size_t(blockIdx.y) * K;
    float acc = 0.f;
    for (int tile0 = 0; tile0 < B; tile0 += kPaperTile) {
        __syncthreads();
        for (int i = threadIdx.x; i < kPaperTile * 24; i += blockDim.x) {
            const int k = tile0 * 24 + i;
            xt[i] = k < K ? __half2float(xb[k]) : 0.f;
        }
        __syncthreads();
        if (row < N) {
            const int end = min(B, tile0 + kPaperTile);
            for (int b = tile0 + lane; b < end; b += 32) {
                int yv[24], m, g;
                decode_file_word(&T, load_file_word(codes + size_t(row) * row_stride, size_t(b)), yv, &m, &g);
                const float* xs = xt + (b - tile0) * 24;
                float dot = 0.f;
#pragma unroll
                for (int j = 0; j < 24; ++j) dot = fmaf(float(yv[j]), xs[j], dot);
                acc = fmaf(gain[g] * T.rsqrt16m[m], dot, acc);
            }
        }
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    if (row < N && lane == 0) {
        float res = row_scales[row] * acc;
        for (int t = 0; t < ntail; ++t)
            res = fmaf(__half2float(tail[size_t(row) * ntail + t]), __half2float(xb[24 * B + t]), res);
        y[size_t(blockIdx.y) * N + row] = res;
    }
}

cudaError_t launch_gemv_paper(const void* codes, size_t row_stride, const float* row_scales, const void* table,
                              const void* x, float* y, int N, int K, int batch, const void* tail, cudaStream_t s) {
    const int ntail = tail ? K % 24 : 0;
    const int B = tail ? K / 24 : (K + 23) / 24;
    dim3 grid((N + 7) / 8, batch);
    k_gemv_paper<<<grid, 256, 0, s>>>(static_cast<const uint8_t*>(codes), row_stride, row_scales,
                                      static_cast<const DeviceTables*>(table), static_cast<const __half*>(x), y, N, K,
                                      B, ntail, static_cast<const __half*>(tail));
    return cudaGetLastError();
}

// ===========================================================================
// Fast kernel
// ===========================================================================
constexpr int kFastThreads = 512;
constexpr int kFastWarps = kFastThreads / 32;
constexpr int kRedStride = 36;                 // floats per row of the transpose buffer (32 + pad)
constexpr int kRowAccFloats = 2048;            // per-CTA buffer of per-(column group, row) sums
constexpr int kXqBytesPerCol = 80;             // 3 planes x 24 bytes, step, sum
constexpr uint32_t kXqHi = 0, kXqMid = 24, kXqLo = 48, kXqStep = 72, kXqSum = 76;

struct FastSmemLayout {
    uint32_t tab, xq, red, rowacc, total;
};
__host__ __device__ inline FastSmemLayout fast_smem_layout(int max_blocks) {
    FastSmemLayout L;
    L.tab = 0;
    L.xq = uint32_t(kFastBytes);
    L.red = L.xq + uint32_t(max_blocks) * kXqBytesPerCol;
    L.rowacc = L.red + kFastWarps * 8 * kRedStride * 4;
    L.total = L.rowacc + kRowAccFloats * 4;
    return L;
}

// Fixed-point image of this matrix's activations in shared memory.  Per block
// column: step = 2^(E-22) with 2^E <= max|x| < 2^(E+1); q_j = rint(x_j / step),
// |q_j| < 2^23, stored as three byte planes (bits 23..16 signed, 15..8 and 7..0
// unsigned), four coordinates per 32-bit word; then the step and sum(q_j).
// A float16 x_j is held exactly when |x_j| >= 2^(E-12); smaller ones are
// rounded to a multiple of the step.  Every CTA does this for itself.
__device__ __forceinline__ void quantise_x(const __half* __restrict__ x, int K, int B, unsigned char* smem,
                                           const FastSmemLayout& L) {
    for (int c = threadIdx.x; c < B; c += blockDim.x) {
        float v[24];
        float mx = 0.f;
#pragma unroll
        for (int j = 0; j < 24; ++j) {
            const int k = 24 * c + j;
            v[j] = k < K ? __half2float(x[k]) : 0.f;
            mx = fmaxf(mx, fabsf(v[j]));
        }
        const uint32_t e = __float_as_uint(mx) >> 23;  // biased exponent of the largest (finite float16 input)
        const float step = mx > 0.f ? __uint_as_float((e - 22u) << 23) : 0.f;
        const float inv = mx > 0.f ? __uint_as_float((276u - e) << 23) : 0.f;
        int sum = 0;
        uint32_t hi[6], mid[6], lo[6];
#pragma unroll
        for (int k = 0; k < 6; ++k) {
            hi[k] = mid[k] = lo[k] = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int q = __float2int_rn(v[4 * k + i] * inv);
                sum += q;
                hi[k] |= (uint32_t(q >> 16) & 0xFFu) << (8 * i);
                mid[k] |= (uint32_t(q >> 8) & 0xFFu) << (8 * i);
                lo[k] |= (uint32_t(q) & 0xFFu) << (8 * i);
            }
        }
        uint32_t* dst = reinterpret_cast<uint32_t*>(smem + L.xq + c * kXqBytesPerCol);
#pragma unroll
        for (int k = 0; k < 6; ++k) {
            dst[k] = hi[k];
            dst[6 + k] = mid[k];
            dst[12 + k] = lo[k];
        }
        reinterpret_cast<float*>(dst)[18] = step;
        reinterpret_cast<int*>(dst)[19] = sum;
    }
}

struct LaneX {
    uint32_t hi[6];   // bits 23..16 of q (signed), int8 x 4
    uint32_t mid[6];  // bits 15..8 (unsigned)
    uint32_t lo[6];   // bits 7..0 (unsigned)
    float step;       // 2^(E-22)
    int sum;          // sum of q over the 24 coordinates
};

// q of one coordinate, read back from the planes in shared memory (fix-up path only).
__device__ __forceinline__ int xq_coord(uint32_t xq_col, int coord) {
    int h;
    uint32_t m, l;
    asm volatile("ld.shared.s8 %0, [%1];" : "=r"(h) : "r"(xq_col + kXqHi + uint32_t(coord)));
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(m) : "r"(xq_col + kXqMid + uint32_t(coord)));
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(l) : "r"(xq_col + kXqLo + uint32_t(coord)));
    return h * 65536 + int(m << 8 | l);
}

// One block: device word -> contribution scale_b * sum_j y_j x_j (Eq. (2) without
// the row scale).  xq_col: shared-memory address of this column's fixed-point image.
template <bool HI>
__device__ __forceinline__ float block_value(uint32_t sm_tab, uint32_t w0, uint32_t w1pair, const LaneX& X,
                                             uint32_t xq_col) {
    FastBlock fb;
    fast_decode<HI>(sm_tab, w0, w1pair, fb);
    int dh = 0, dm = 0, dl = 0, n2 = 0, n1 = 0;
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        dh = dp4a_ss(fb.y0[k], X.hi[k], dh);
        dm = dp4a_su(fb.y0[k], X.mid[k], dm);
        dl = dp4a_su(fb.y0[k], X.lo[k], dl);
        n2 = dp4a_ss(fb.y0[k], fb.y0[k], n2);
        n1 = dp4a_ss(fb.y0[k], 0x01010101u, n1);
    }
    // |sum_j y_j q_j| <= sqrt(24 * 416) * 2^23 < 2^31: the block's dot product is an exact int32
    int dot = dh * 65536 + (dm * 256 + dl);
    if (fb.flags1 | fb.flags3) {  // a coordinate of rank 4: about 1.6 % of uniform random words
        if (fb.flags1) {
            int j, dy, dsq;
            rank4_fix(fb.flags1, fb.sel1, &j, &dy, &dsq);
            dot += dy * xq_coord(xq_col, j);
            n2 += dsq;
            n1 += dy;
        }
        if (fb.flags3) {
            int j, dy, dsq;
            rank4_fix(fb.flags3, fb.sel3, &j, &dy, &dsq);
            dot += dy * xq_coord(xq_col, 16 + j);
            n2 += dsq;
            n1 += dy;
        }
    }
    if (fb.p13) {  // p = 1: y = 1 - y0
        dot = X.sum - dot;
        n2 = n2 - 2 * n1 + 24;
    }
    // n2 = 16 m; the scale table holds gain[g] / sqrt(16 m) at byte 128 g + 4 m
    const float scale = lds32f(sm_tab + kSmScale + fb.goff + (uint32_t(n2) >> 2));
    return float(dot) * (scale * X.step);
}

__global__ void __launch_bounds__(kFastThreads, 1)
k_gemv_fast(const DeviceTables* __restrict__ tab, const Problem* __restrict__ problems, const Problem single,
            int count, int batch, int max_blocks) {
    extern __shared__ __align__(16) unsigned char smem[];
    const FastSmemLayout L = fast_smem_layout(max_blocks);
    stage_fast_tables(tab, reinterpret_cast<uint4*>(smem));
    const uint32_t sm_tab = smem_u32(smem);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* red = reinterpret_cast<float*>(smem + L.red) + warp * 8 * kRedStride;
    float* rowacc = reinterpret_cast<float*>(smem + L.rowacc);

    const int njobs = problems ? count : batch;
    for (int job = 0; job < njobs; ++job) {
        Problem P = problems ? problems[job] : single;
        if (!problems) {  // batch column `job` of the single product
            P.x = static_cast<const __half*>(P.x) + size_t(job) * P.K;
            P.y = P.y + size_t(job) * P.N;
        }
        const int ntail = P.tail ? P.K % 24 : 0;
        const int B = P.tail ? P.K / 24 : (P.K + 23) / 24;
        const int groups = (P.N + 7) / 8;
        const int g_begin = int((long long)blockIdx.x * groups / gridDim.x);
        const int g_end = int((long long)(blockIdx.x + 1) * groups / gridDim.x);
        const int CG = (B + 31) / 32;
        __syncthreads();  // previous job's epilogue is done with xq / rowacc; tables are staged
        if (g_begin < g_end) quantise_x(static_cast<const __half*>(P.x), P.K, B, smem, L);
        __syncthreads();

        const bool narrow = CG <= kFastWarps;
        const int RL = narrow ? kFastWarps / CG : 1;  // warps sharing a column group walk different rows
        const int rl = narrow ? warp / CG : 0;
        const int cg_step = narrow ? CG : kFastWarps;
        // rows of this CTA are processed in chunks whose per-(column group, row) sums fit the buffer
        const int chunk_groups = max(1, kRowAccFloats / (8 * CG));
        const uint4* codes = static_cast<const uint4*>(P.codes);

        for (int c_begin = g_begin; c_begin < g_end; c_begin += chunk_groups) {
            const int c_end = min(g_end, c_begin + chunk_groups);
            const int rows_chunk = (c_end - c_begin) * 8;
            if (rl < RL) {
                for (int cg = narrow ? warp % CG : warp; cg < CG; cg += cg_step) {
                    const int col = cg * 32 + lane;
                    const bool active = col < B;
                    const uint32_t xq_col = sm_tab + L.xq + uint32_t(active ? col : 0) * kXqBytesPerCol;
                    LaneX X;
                    {
                        uint32_t q[20];
#pragma unroll
                        for (int k = 0; k < 5; ++k)
                            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(q[4 * k]), "=r"(q[4 * k + 1]), "=r"(q[4 * k + 2]), "=r"(q[4 * k + 3])
                                         : "r"(xq_col + 16u * k));
#pragma unroll
                        for (int k = 0; k < 6; ++k) {
                            X.hi[k] = active ? q[k] : 0u;
                            X.mid[k] = active ? q[6 + k] : 0u;
                            X.lo[k] = active ? q[12 + k] : 0u;
                        }
                        X.step = active ? __uint_as_float(q[18]) : 0.f;
                        X.sum = active ? int(q[19]) : 0;
                    }
                    const uint4 zero4 = make_uint4(0, 0, 0, 0);
                    int g = c_begin + rl;
                    uint4 n0 = zero4, n1 = zero4, n2 = zero4;
                    if (g < c_end && active) {
                        const uint4* rec = codes + size_t(g) * 3 * B + col;
                        n0 = __ldg(rec); n1 = __ldg(rec + B); n2 = __ldg(rec + 2 * size_t(B));
                    }
                    for (; g < c_end; g += RL) {
                        const uint4 a = n0, b = n1, h = n2;
                        if (g + RL < c_end && active) {  // prefetch the next record
                            const uint4* rec = codes + size_t(g + RL) * 3 * B + col;
                            n0 = __ldg(rec); n1 = __ldg(rec + B); n2 = __ldg(rec + 2 * size_t(B));
                        }
                        float v[8];
                        v[0] = block_value<false>(sm_tab, a.x, h.x, X, xq_col);
                        v[1] = block_value<true>(sm_tab, a.y, h.x, X, xq_col);
                        v[2] = block_value<false>(sm_tab, a.z, h.y, X, xq_col);
                        v[3] = block_value<true>(sm_tab, a.w, h.y, X, xq_col);
                        v[4] = block_value<false>(sm_tab, b.x, h.z, X, xq_col);
                        v[5] = block_value<true>(sm_tab, b.y, h.z, X, xq_col);
                        v[6] = block_value<false>(sm_tab, b.z, h.w, X, xq_col);
                        v[7] = block_value<true>(sm_tab, b.w, h.w, X, xq_col);
                        // transpose through shared memory: lane l then owns row l/4, lanes 8(l%4)..8(l%4)+7
                        __syncwarp();
#pragma unroll
                        for (int r = 0; r < 8; ++r) red[r * kRedStride + lane] = v[r];
                        __syncwarp();
                        const float4 s0 = *reinterpret_cast<const float4*>(red + (lane >> 2) * kRedStride + 8 * (lane & 3));
                        const float4 s1 = *reinterpret_cast<const float4*>(red + (lane >> 2) * kRedStride + 8 * (lane & 3) + 4);
                        float sum = ((s0.x + s0.y) + (s0.z + s0.w)) + ((s1.x + s1.y) + (s1.z + s1.w));
                        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
                        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
                        if ((lane & 3) == 0) rowacc[cg * rows_chunk + (g - c_begin) * 8 + (lane >> 2)] = sum;
                    }
                }
            }
            __syncthreads();
            // epilogue: sum the column groups in a fixed order, row scale, tail (Sec. 5.1)
            for (int t = threadIdx.x; t < rows_chunk; t += blockDim.x) {
                const int row = c_begin * 8 + t;
                if (row >= P.N) continue;
                float acc = 0.f;
                for (int cg = 0; cg < CG; ++cg) acc += rowacc[cg * rows_chunk + t];
                float res = P.row_scales[row] * acc;
                const __half* xh = static_cast<const __half*>(P.x);
                const __half* tl = static_cast<const __half*>(P.tail);
                for (int k = 0; k < ntail; ++k)
                    res = fmaf(__half2float(tl[size_t(row) * ntail + k]), __half2float(xh[24 * B + k]), res);
                P.y[row] = res;
            }
            __syncthreads();
        }
    }
}

cudaError_t launch_gemv_fast(const Problem& single, int batch, const Problem* problems_dev, int count, int max_blocks,
                             const void* table, cudaStream_t s) {
    static int num_sms[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && num_sms[dev] == 0) {
        int n = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(k_gemv_fast, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        num_sms[dev] = n;
    }
    const int sms = dev < 64 ? num_sms[dev] : 148;
    const FastSmemLayout L = fast_smem_layout(max_blocks);
    if (L.total > 227u * 1024u) return cudaErrorInvalidValue;
    int grid = sms;
    if (!problems_dev) {
        const int groups = (single.N + 7) / 8;
        if (groups < grid) grid = groups;
    }
    k_gemv_fast<<<grid, kFastThreads, L.total, s>>>(static_cast<const DeviceTables*>(table), problems_dev, single,
                                                    count, batch, max_blocks);
    return cudaGetLastError();
}

}  // namespace tetra
