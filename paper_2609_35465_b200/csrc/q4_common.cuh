// Pieces shared by the kernels of the 4-bit group-quantised format (Sec. 4.1, 4.4, 5.1): the packed
// layout's chunk size, the nibble-to-float16 operand trick, and small PTX wrappers.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace tetra {
namespace {

// Packed layout.  Rows are taken in strips of 32, columns in groups of G; the data of (strip, group) is one
// contiguous chunk of CH = (G / 64) * 1024 + 128 bytes at (strip * groups + group) * CH:
//   for each 64-column tile j of the group, two 512-byte sub-tiles h = 0, 1 (rows 16 h .. 16 h + 15 of the
//   strip) at j * 1024 + h * 512, in which lane = 4 g + t of a warp owns 16 bytes = four words m = 0..3; word m
//   holds, as nibbles n0..n7 (n_i at bits 4 i), the weights of columns c = 64 j + 16 t + 4 m + {0,1,2,3}:
//       n0, n4 = row g,     c + 0, c + 1        n1, n5 = row g,     c + 2, c + 3
//       n2, n6 = row g + 8, c + 0, c + 1        n3, n7 = row g + 8, c + 2, c + 3      (rows within the sub-tile)
//   then 32 (scale, offset) float16 pairs, one per row of the strip.
// A warp streams whole chunks; nothing else of the matrix is read.
__host__ __device__ constexpr int q4_chunk_bytes(int G) { return (G / 64) * 1024 + 128; }

__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// (a, a) * (b0, b1) + (c0, c1) in one instruction (fma.rn.f32x2).
__device__ __forceinline__ void fma2(float a, float b0, float b1, float& c0, float& c1) {
    uint64_t aa, bb, cc;
    asm("mov.b64 %0, {%1, %1};" : "=l"(aa) : "f"(a));
    asm("mov.b64 %0, {%1, %2};" : "=l"(bb) : "f"(b0), "f"(b1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(cc) : "f"(c0), "f"(c1));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(cc) : "l"(aa), "l"(bb));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(c0), "=f"(c1) : "l"(cc));
}

__device__ __forceinline__ uint32_t lop_and_or(uint32_t a, uint32_t mask, uint32_t magic) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(magic));  // (a & mask) | magic
    return r;
}
__device__ __forceinline__ void q4_lds128(uint32_t saddr, uint32_t (&v)[4]) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(saddr));
}
__device__ __forceinline__ void q4_cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
template <int PENDING>
__device__ __forceinline__ void q4_cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
}

// First MMA of a group: the accumulator starts from c (minus the group's bias sums).
__device__ __forceinline__ void mma_f16_first(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, float c_even,
                                              float c_odd) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%10,%11};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c_even), "f"(c_odd));
}


}  // namespace
}  // namespace tetra
