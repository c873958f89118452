// Pieces shared by the decode-and-multiply kernels: the lane's activation record, the per-block
// product, the warp's transpose reduction, and the launch helpers.
#pragma once
#include <cuda_fp16.h>

#include "tetra_device.cuh"
#include "tetra_launch.h"

namespace tetra {

constexpr int kRedStride = 36;                 // floats per row of the transpose buffer (32 + pad)
constexpr int kRedFloats = 8 * kRedStride;     // per warp
constexpr int kXqBytesPerCol = 80;             // 3 planes x 24 bytes, step, sum

struct LaneX {
    uint32_t hi[6];   // bits 23..16 of q (signed), int8 x 4
    uint32_t mid[6];  // bits 15..8 (unsigned)
    uint32_t lo[6];   // bits 7..0 (unsigned)
    float step;       // 2^(E-22)
    int sum;          // sum of q over the 24 coordinates (kept in the record; unused by the kernels)
};

__device__ __forceinline__ void lane_x_from_words(const uint32_t q[20], bool active, LaneX& X) {
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        X.hi[k] = active ? q[k] : 0u;
        X.mid[k] = active ? q[6 + k] : 0u;
        X.lo[k] = active ? q[12 + k] : 0u;
    }
    X.step = active ? __uint_as_float(q[18]) : 0.f;
    X.sum = active ? int(q[19]) : 0;
}

// One block: device word -> contribution scale_b * sum_j y_j x_j (Eq. (2) without
// the row scale).
template <bool HI>
__device__ __forceinline__ float block_value(uint32_t sm_tab, uint32_t w0, uint32_t w1pair, const LaneX& X,
                                             float addend = 0.f) {
    FastBlock fb;
    fast_decode<HI>(sm_tab, w0, w1pair, fb);
    // The squared norm 16 m is accumulated on top of the address of the gain's half of the scale table:
    // that table holds -gain[g] / sqrt(16 m) at 512 g + 16 m, so the sum IS the address of the scale
    // (16 m <= 416 for every word, Sec. 3.4, so it stays inside the table's half).
    int dh = 0, dm = 0, dl = 0, n2 = int(fb.goff);
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        dh = dp4a_ss(fb.y[k], X.hi[k], dh);
        dm = dp4a_su(fb.y[k], X.mid[k], dm);
        dl = dp4a_su(fb.y[k], X.lo[k], dl);
        n2 = dp4a_ss(fb.y[k], fb.y[k], n2);
    }
    // |sum_j y_j q_j| <= sqrt(24 * 416) * 2^23 < 2^31: the block's dot product is an exact int32
    // (of -y: the scale carries the other minus sign)
    int dot = dh * 65536 + (dm * 256 + dl);
    const float scale = lds32f(uint32_t(n2));
    return fmaf(float(dot), scale * X.step, addend);  // addend: the caller's running sum (one FFMA)
}

// The eight blocks of one 48-byte record (rows 8G..8G+7 of one column).
__device__ __forceinline__ void record_values(uint32_t sm_tab, const uint4& a, const uint4& b, const uint4& h,
                                              const LaneX& X, float v[8]) {
    v[0] = block_value<false>(sm_tab, a.x, h.x, X);
    v[1] = block_value<true>(sm_tab, a.y, h.x, X);
    v[2] = block_value<false>(sm_tab, a.z, h.y, X);
    v[3] = block_value<true>(sm_tab, a.w, h.y, X);
    v[4] = block_value<false>(sm_tab, b.x, h.z, X);
    v[5] = block_value<true>(sm_tab, b.y, h.z, X);
    v[6] = block_value<false>(sm_tab, b.z, h.w, X);
    v[7] = block_value<true>(sm_tab, b.w, h.w, X);
}

// The same, added to the caller's eight running sums.
__device__ __forceinline__ void record_accumulate(uint32_t sm_tab, const uint4& a, const uint4& b, const uint4& h,
                                                  const LaneX& X, float acc[8]) {
    acc[0] = block_value<false>(sm_tab, a.x, h.x, X, acc[0]);
    acc[1] = block_value<true>(sm_tab, a.y, h.x, X, acc[1]);
    acc[2] = block_value<false>(sm_tab, a.z, h.y, X, acc[2]);
    acc[3] = block_value<true>(sm_tab, a.w, h.y, X, acc[3]);
    acc[4] = block_value<false>(sm_tab, b.x, h.z, X, acc[4]);
    acc[5] = block_value<true>(sm_tab, b.y, h.z, X, acc[5]);
    acc[6] = block_value<false>(sm_tab, b.z, h.w, X, acc[6]);
    acc[7] = block_value<true>(sm_tab, b.w, h.w, X, acc[7]);
}

// Sums v[r] over the 32 lanes for r = 0..7 through the warp's shared-memory
// buffer.  Afterwards lane l holds, for row l / 4, the partial sum over lanes
// 8 (l % 4) .. 8 (l % 4) + 7; the caller finishes with two shuffles.
__device__ __forceinline__ float transpose_partial(float* red, int lane, const float v[8]) {
    __syncwarp();
#pragma unroll
    for (int r = 0; r < 8; ++r) red[r * kRedStride + lane] = v[r];
    __syncwarp();
    const float4 s0 = *reinterpret_cast<const float4*>(red + (lane >> 2) * kRedStride + 8 * (lane & 3));
    const float4 s1 = *reinterpret_cast<const float4*>(red + (lane >> 2) * kRedStride + 8 * (lane & 3) + 4);
    return ((s0.x + s0.y) + (s0.z + s0.w)) + ((s1.x + s1.y) + (s1.z + s1.w));
}

// Launch with programmatic stream serialization allowed: the kernel may start while its predecessor
// in the stream is still running and synchronises with it through pdl_wait().
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid));
    cfg.blockDim = dim3(unsigned(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}


}  // namespace tetra
