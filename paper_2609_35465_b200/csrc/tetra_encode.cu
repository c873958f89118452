// Encoder search (Sec. 3.1, Eq. (2)): for a block of 24 weights, the point of the format's codebook whose
// direction is closest to the block, and the gain bit.
//
// The paper's own search is not exhaustive and runs on a CPU; this kernel computes the exact optimum of the
// same objective,  max <w, y> / (|w| |y|)  over all 2^47 indices, by using what the format's structure gives:
//   * a section's coordinates depend on (parity p, pattern byte c, rank row) only, the pattern bytes of all
//     three sections are the 128 even-weight bytes, and for fixed (p, c, class) the section's squared norm is
//     16 k + r with r fixed by (p, weight of c, class) and k = 0..9: per section, byte and class only ten best
//     correlations matter (one per k);
//   * the sections are tied by the trellis path, by the parity and by Eq. (3) (r3 = p ^ r ^ delta): they are
//     joined state by state with the summed norm and the class parity as extra state.
// One CTA of 384 threads works on one block at a time: three groups of 128 threads, one per section, thread =
// pattern byte.  For every batch of 32 rank rows a group tabulates, per row, the partial correlations and
// norms of the 16 patterns of each half of the byte (so a (row, byte) candidate costs two shared loads and two
// additions) while every thread scans the batch before for its own byte and keeps the best correlation per
// (class, k) in a private column of shared memory (no atomics; two columns, for even and odd rows, so that
// two updates are in flight).  The join runs on the same CTA, every thread gathering a few entries of the
// second cut; the rows that attain the winning entries are found by a second scan of three lists.
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/tetra.h"
#include "tetra_device.cuh"
#include "tetra_launch.h"
#include "tetra_tables.h"

namespace tetra {
namespace {

constexpr int kEncThreads = 384;
constexpr int kEncBatch = 32;       // rank rows per batch
constexpr int kEncStride = 33;      // row-table entries are 33 rows apart (bank spread)
constexpr float kNeg = -1.0e30f;
constexpr float kNegTest = -1.0e29f;

struct EncShared {
    uint32_t rows[4096];
    uint16_t branches[1024];
    uint8_t prefixes[128];
    uint8_t suffixes[128];
    uint16_t incoming[64][16];                 // per state after the branch: s8 | b2 << 6
    int incoming_count[64];
    float A[3][8][4][8];                       // w_j * value(o, rank)
    int V2[4][8];                              // value(o, rank)^2
    uint2 rowtab[2][3][32 * kEncStride];       // two buffers of (partial correlation, partial norm): entry (half * 16 + pattern), row
    float T[3][2][20][128];                    // best correlation per (class * 10 + k), byte; one copy for even, one for odd rows
    float F1[64][2][20];                       // after section 1: state, class, norm / 8
    float H[39][128];                          // after section 2: norm / 8, (state after the branch) * 2 + class parity
    float red_val[kEncThreads / 32];
    uint32_t red_arg[kEncThreads / 32];
    float w[24];
    // best so far
    float best_val, best_corr;
    int best_norm;
    uint32_t best_path;                        // s8 | b1 << 6 | b2 << 7 | b3 << 11 | p << 12 | r << 13
    int best_field[3];
    int found_field[3];
};

__device__ __forceinline__ int even_byte(int ci) {  // the 128 even-weight bytes, by index
    const int h = ci >> 3, li = ci & 7;
    return (h << 4) | (li << 1) | ((__popc(li) ^ __popc(h)) & 1);
}
__device__ __forceinline__ int even_index(int byte) { return ((byte >> 4) << 3) | ((byte & 15) >> 1); }
// squared norm of a section = 16 k + residue
__device__ __forceinline__ int norm_residue(int p, int cls, int byte) { return p ? (cls ? 0 : 8) : ((4 * __popc(byte)) & 15); }

__device__ __forceinline__ void group_barrier(int group) {
    asm volatile("bar.sync %0, 128;" ::"r"(1 + group) : "memory");
}

// Rows of a section's list for a class: sections 0 and 2 read all 2048 rows of the class, the middle section
// the first 1240 (class 0) or 808 (class 1) of them (Sec. 3.3).
__device__ __forceinline__ int list_length(int section, int cls) {
    return section == 1 ? (cls ? 2048 - kMiddleClass0 : kMiddleClass0) : 2048;
}

// Largest value over the CTA with its argument; ties go to the smaller argument.  Everyone gets the result.
__device__ void cta_argmax(EncShared& S, float& val, uint32_t& arg) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        const float v2 = __shfl_xor_sync(0xFFFFFFFFu, val, o);
        const uint32_t a2 = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
        if (v2 > val || (v2 == val && a2 < arg)) {
            val = v2;
            arg = a2;
        }
    }
    __syncthreads();
    if (lane == 0) {
        S.red_val[warp] = val;
        S.red_arg[warp] = arg;
    }
    __syncthreads();
    val = S.red_val[0];
    arg = S.red_arg[0];
    for (int k = 1; k < kEncThreads / 32; ++k) {
        const float v2 = S.red_val[k];
        const uint32_t a2 = S.red_arg[k];
        if (v2 > val || (v2 == val && a2 < arg)) {
            val = v2;
            arg = a2;
        }
    }
}

__global__ void __launch_bounds__(kEncThreads, 1)
k_encode(const float* __restrict__ w, const float* __restrict__ sigma, const DeviceTables* __restrict__ tab,
         unsigned char* __restrict__ codes, float* __restrict__ cosine, size_t nblocks) {
    extern __shared__ __align__(16) unsigned char enc_smem[];
    EncShared& S = *reinterpret_cast<EncShared*>(enc_smem);
    const int tid = threadIdx.x;
    const int sg = tid >> 7, ct = tid & 127;  // section group, pattern-byte index
    // --- tables, once per CTA ---
    for (int i = tid; i < 4096; i += kEncThreads) S.rows[i] = tab->paper.rows[i];
    for (int i = tid; i < 1024; i += kEncThreads) S.branches[i] = tab->paper.branches[i];
    if (tid < 128) {
        S.prefixes[tid] = tab->paper.prefixes[tid];
        S.suffixes[tid] = tab->paper.suffixes[tid];
    }
    if (tid < 64) S.incoming_count[tid] = 0;
    if (tid < 32) S.V2[tid >> 3][tid & 7] = rank_value(tid >> 3, tid & 7) * rank_value(tid >> 3, tid & 7);
    __syncthreads();
    for (int i = tid; i < 1024; i += kEncThreads) {  // order within a state's list does not matter for the maximum,
        const int s16 = S.branches[i] >> 8;          // but it decides ties: sort below
        const int slot = atomicAdd(&S.incoming_count[s16], 1);
        if (slot < 16) S.incoming[s16][slot] = uint16_t(i);  // i = 16 s8 + b2
    }
    __syncthreads();
    if (tid < 64) {  // insertion sort of 16 entries: the same order in every CTA and run
        for (int a = 1; a < 16; ++a) {
            const uint16_t v = S.incoming[tid][a];
            int b = a - 1;
            while (b >= 0 && S.incoming[tid][b] > v) {
                S.incoming[tid][b + 1] = S.incoming[tid][b];
                --b;
            }
            S.incoming[tid][b + 1] = v;
        }
    }
    const float gain0 = tab->gain[0], gain1 = tab->gain[1];
    const int my_byte = even_byte(ct);
    const int my_lo = my_byte & 15, my_hi = my_byte >> 4;
    __syncthreads();

    for (size_t block = blockIdx.x; block < nblocks; block += gridDim.x) {
        if (tid < 24) S.w[tid] = w[block * 24 + tid];
        if (tid == 0) {
            S.best_val = kNeg;
            S.best_corr = 0.f;
            S.best_norm = 0;
            S.best_path = 0;
            S.best_field[0] = S.best_field[1] = S.best_field[2] = 0;
        }
        __syncthreads();
        for (int i = tid; i < 3 * 8 * 4 * 8; i += kEncThreads) {
            const int rho = i & 7, o = (i >> 3) & 3, j = (i >> 5) & 7, s = i >> 8;
            S.A[s][j][o][rho] = S.w[8 * s + j] * float(rank_value(o, rho));
        }
        float wn2 = 0.f;
#pragma unroll
        for (int j = 0; j < 24; ++j) wn2 = fmaf(S.w[j], S.w[j], wn2);
        __syncthreads();
        if (wn2 == 0.f) {  // a zero block encodes as the all-zero word
            if (tid < 6) codes[block * 6 + tid] = 0;
            if (tid == 0 && cosine) cosine[block] = 0.f;
            continue;
        }

        for (int p = 0; p < 2; ++p) {
            // ---------------- section tables ----------------
            for (int i = ct; i < 2 * 20 * 128; i += 128) (&S.T[sg][0][0][0])[i] = kNeg;
            // thread (row of the batch = ct / 2, half of the byte = ct & 1) tabulates 16 patterns while the whole
            // group scans the batch before: one barrier per batch
            auto produce = [&](int buf, int cls, int b0) {
                const int len = list_length(sg, cls);
                const int r = ct >> 1, half = ct & 1;
                if (ct < 2 * kEncBatch && b0 + r < len) {
                    const uint32_t rw = S.rows[2048 * cls + b0 + r];
                    float P[16];
                    int Nn[16];
                    P[0] = 0.f;
                    Nn[0] = 0;
                    float d[4];
                    int dn[4];
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const int j = 4 * half + jj, rho = (rw >> (4 * j)) & 7;
                        const float a0 = S.A[sg][j][p][rho], a1 = S.A[sg][j][p + 2][rho];
                        const int n0 = S.V2[p][rho], n1 = S.V2[p + 2][rho];
                        P[0] += a0;
                        Nn[0] += n0;
                        d[jj] = a1 - a0;
                        dn[jj] = n1 - n0;
                    }
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj)
#pragma unroll
                        for (int m = 0; m < (1 << jj); ++m) {
                            P[m | (1 << jj)] = P[m] + d[jj];
                            Nn[m | (1 << jj)] = Nn[m] + dn[jj];
                        }
#pragma unroll
                    for (int m = 0; m < 16; ++m)
                        S.rowtab[buf][sg][(half * 16 + m) * kEncStride + r] = make_uint2(__float_as_uint(P[m]), uint32_t(Nn[m]) * 32u);
                }
            };
            // the batches of both classes as one sequence
            const int nb0 = (list_length(sg, 0) + kEncBatch - 1) / kEncBatch, nb1 = (list_length(sg, 1) + kEncBatch - 1) / kEncBatch;
            produce(0, 0, 0);
            group_barrier(sg);
            for (int bi = 0; bi < nb0 + nb1; ++bi) {
                const int buf = bi & 1;
                const int cls = bi < nb0 ? 0 : 1, b0 = (bi < nb0 ? bi : bi - nb0) * kEncBatch;
                if (bi + 1 < nb0 + nb1) {
                    const int nbi = bi + 1;
                    produce(buf ^ 1, nbi < nb0 ? 0 : 1, (nbi < nb0 ? nbi : nbi - nb0) * kEncBatch);
                }
                const int nb = min(kEncBatch, list_length(sg, cls) - b0);
                const uint2* lo_tab = &S.rowtab[buf][sg][my_lo * kEncStride];
                const uint2* hi_tab = &S.rowtab[buf][sg][(16 + my_hi) * kEncStride];
                // a candidate's cell: the tables hold 32 x norm, a column's cells are 512 bytes apart and the norm is
                // 16 k + residue, so  cell = column + 32 norm - 32 residue  (one three-input addition)
                const uint32_t res32 = uint32_t(norm_residue(p, cls, my_byte)) * 32u;
                const uint32_t t_even = smem_u32(&S.T[sg][0][cls * 10][ct]) - res32;
                const uint32_t t_odd = smem_u32(&S.T[sg][1][cls * 10][ct]) - res32;
                auto update = [&](uint32_t column, uint2 lo, uint2 hi) {
                    const uint32_t cell = column + lo.y + hi.y;
                    float v;
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(cell));
                    v = fmaxf(v, __uint_as_float(lo.x) + __uint_as_float(hi.x));
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(cell), "f"(v) : "memory");
                };
                // At odd parity every coordinate is +-(2 rank + 1) whatever the pattern byte, so a row's norm is its
                // cost and the rows of a class come sorted by cost: nearly every batch has ONE norm, the same for
                // all bytes, and its best correlation is a running maximum in a register.
                const uint32_t n_first = lo_tab[0].y + hi_tab[0].y, n_last = lo_tab[nb - 1].y + hi_tab[nb - 1].y;
                if (p == 1 && nb == kEncBatch && n_first == n_last) {
                    float m0 = kNeg, m1 = kNeg;
#pragma unroll
                    for (int r = 0; r < kEncBatch; r += 2) {
                        m0 = fmaxf(m0, __uint_as_float(lo_tab[r].x) + __uint_as_float(hi_tab[r].x));
                        m1 = fmaxf(m1, __uint_as_float(lo_tab[r + 1].x) + __uint_as_float(hi_tab[r + 1].x));
                    }
                    const uint32_t cell = t_even + n_first;
                    float v;
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(cell));
                    v = fmaxf(v, fmaxf(m0, m1));
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(cell), "f"(v) : "memory");
                } else if (nb == kEncBatch) {
#pragma unroll
                    for (int r = 0; r < kEncBatch; r += 2) {  // two independent read-modify-write chains, loads first
                        const uint2 lo0 = lo_tab[r], hi0 = hi_tab[r], lo1 = lo_tab[r + 1], hi1 = hi_tab[r + 1];
                        const uint32_t cell0 = t_even + lo0.y + hi0.y, cell1 = t_odd + lo1.y + hi1.y;
                        float v0, v1;
                        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v0) : "r"(cell0));
                        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v1) : "r"(cell1));
                        v0 = fmaxf(v0, __uint_as_float(lo0.x) + __uint_as_float(hi0.x));
                        v1 = fmaxf(v1, __uint_as_float(lo1.x) + __uint_as_float(hi1.x));
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(cell0), "f"(v0) : "memory");
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(cell1), "f"(v1) : "memory");
                    }
                } else {
                    for (int r = 0; r < nb; ++r) update(t_even, lo_tab[r], hi_tab[r]);
                }
                group_barrier(sg);
            }
            for (int i = ct; i < 20 * 128; i += 128)  // fold the odd rows' copy into the even rows'
                (&S.T[sg][0][0][0])[i] = fmaxf((&S.T[sg][0][0][0])[i], (&S.T[sg][1][0][0])[i]);
            __syncthreads();

            // ---------------- join: first cut ----------------
            for (int e = tid; e < 64 * 2 * 20; e += kEncThreads) {
                const int n8 = e % 20, cls = (e / 20) & 1, s8 = e / 40;
                float best = kNeg;
#pragma unroll
                for (int b1 = 0; b1 < 2; ++b1) {
                    const int byte = S.prefixes[2 * s8 + b1];
                    const int rem = 8 * n8 - norm_residue(p, cls, byte);
                    if (rem >= 0 && (rem & 15) == 0 && (rem >> 4) < 10) best = fmaxf(best, S.T[0][0][cls * 10 + (rem >> 4)][even_index(byte)]);
                }
                S.F1[s8][cls][n8] = best;
            }
            __syncthreads();
            // ---------------- second cut ----------------
            // thread = (state after the branch, class parity): all 39 entries of its column are accumulated in
            // registers (two sets, for the two possible norm residues of section 2's byte) over the 16 branches
            // into the state, the class of section 1, the 20 norms after section 1 and the 10 of section 2
            if (tid < 128) {
                const int s16 = tid >> 1, par = tid & 1;
                float h0[38], h1[38];  // index n8 + 2 k2, residue 0 / 8 of section 2
#pragma unroll
                for (int i = 0; i < 38; ++i) h0[i] = h1[i] = kNeg;
                for (int in = 0; in < 16; ++in) {
                    const int sb = S.incoming[s16][in], s8 = sb >> 4;
                    const int byte2 = S.branches[sb] & 0xFF, ci2 = even_index(byte2);
                    for (int cls1 = 0; cls1 < 2; ++cls1) {
                        const int cls2 = par ^ cls1;
                        float a[20], b[10];
#pragma unroll
                        for (int n8 = 0; n8 < 20; ++n8) a[n8] = S.F1[s8][cls1][n8];
#pragma unroll
                        for (int k2 = 0; k2 < 10; ++k2) b[k2] = S.T[1][0][cls2 * 10 + k2][ci2];
                        if (norm_residue(p, cls2, byte2)) {
#pragma unroll
                            for (int n8 = 0; n8 < 20; ++n8)
#pragma unroll
                                for (int k2 = 0; k2 < 10; ++k2) h1[n8 + 2 * k2] = fmaxf(h1[n8 + 2 * k2], a[n8] + b[k2]);
                        } else {
#pragma unroll
                            for (int n8 = 0; n8 < 20; ++n8)
#pragma unroll
                                for (int k2 = 0; k2 < 10; ++k2) h0[n8 + 2 * k2] = fmaxf(h0[n8 + 2 * k2], a[n8] + b[k2]);
                        }
                    }
                }
                // an absent entry stays far below every real one (sums of two absent entries are more negative still)
#pragma unroll
                for (int q = 0; q < 39; ++q) {
                    float v = q < 38 ? h0[q] : kNeg;
                    if (q >= 1) v = fmaxf(v, h1[q - 1]);
                    S.H[q][tid] = v > kNegTest ? v : kNeg;
                }
            }
            __syncthreads();
            // ---------------- last section and the objective ----------------
            float val = kNeg;
            uint32_t arg = 0xFFFFFFFFu;
            if (tid < 256) {
                const int s16 = tid >> 2, b3 = (tid >> 1) & 1, par = tid & 1;
                const int byte3 = S.suffixes[2 * s16 + b3], ci3 = even_index(byte3);
                const int cls3 = p ^ par, res3 = norm_residue(p, cls3, byte3);
                for (int q = 0; q < 39; ++q) {
                    const float a = S.H[q][s16 * 2 + par];
                    if (a < kNegTest) continue;
#pragma unroll
                    for (int k3 = 0; k3 < 10; ++k3) {
                        const float b = S.T[2][0][cls3 * 10 + k3][ci3];
                        const int n = 8 * q + 16 * k3 + res3;
                        if (b > kNegTest && n > 0) {
                            const float v = (a + b) / sqrtf(float(n));
                            const uint32_t code = (uint32_t(tid) << 16) | (uint32_t(q) << 8) | uint32_t(k3);
                            if (v > val || (v == val && code < arg)) {
                                val = v;
                                arg = code;
                            }
                        }
                    }
                }
            }
            cta_argmax(S, val, arg);
            if (val > S.best_val) {  // uniform: resolve the path and the rows while this parity's tables are alive
                const int wt = int(arg >> 16), q = int(arg >> 8) & 0xFF, k3 = int(arg & 0xFF);
                const int s16 = wt >> 2, b3 = (wt >> 1) & 1, par = wt & 1;
                // which branch, class and norms attain the winning entry of the second cut: the first, in (branch,
                // class, norm) order, whose sum is the entry (the same additions as above, so the match is exact)
                uint32_t back = 0;
                {
                    const float target = S.H[q][s16 * 2 + par];
                    bool found = false;
                    for (int in = 0; in < 16 && !found; ++in) {
                        const int sb = S.incoming[s16][in], s8c = sb >> 4, b2c = sb & 15;
                        const int byte2 = S.branches[sb] & 0xFF, ci2 = even_index(byte2);
                        for (int c1 = 0; c1 < 2 && !found; ++c1) {
                            const int c2 = par ^ c1, res2 = norm_residue(p, c2, byte2) >> 3;
                            for (int kk = 0; kk < 10 && !found; ++kk) {
                                const int n8c = q - 2 * kk - res2;
                                if (n8c < 0 || n8c >= 20) continue;
                                if (S.F1[s8c][c1][n8c] + S.T[1][0][c2 * 10 + kk][ci2] == target) {
                                    back = uint32_t(s8c) | (uint32_t(b2c) << 6) | (uint32_t(c1) << 10) |
                                           (uint32_t(n8c) << 11) | (uint32_t(kk) << 16);
                                    found = true;
                                }
                            }
                        }
                    }
                }
                const int s8 = back & 63, b2 = (back >> 6) & 15, cls1 = (back >> 10) & 1, n8 = (back >> 11) & 31,
                          k2 = (back >> 16) & 15;
                const int cls2 = par ^ cls1, cls3 = p ^ par;
                // the prefix that attains F1
                int b1 = 0, k1 = 0;
                {
                    float bestv = kNeg;
                    for (int bb = 0; bb < 2; ++bb) {
                        const int byte = S.prefixes[2 * s8 + bb];
                        const int rem = 8 * n8 - norm_residue(p, cls1, byte);
                        if (rem >= 0 && (rem & 15) == 0 && (rem >> 4) < 10) {
                            const float v = S.T[0][0][cls1 * 10 + (rem >> 4)][even_index(byte)];
                            if (v > bestv) {
                                bestv = v;
                                b1 = bb;
                                k1 = rem >> 4;
                            }
                        }
                    }
                }
                const int bytes[3] = {S.prefixes[2 * s8 + b1], S.branches[16 * s8 + b2] & 0xFF, S.suffixes[2 * s16 + b3]};
                const int clss[3] = {cls1, cls2, cls3};
                const int ks[3] = {k1, k2, k3};
                // second scan: group sg looks for the row of section sg (largest correlation at that byte, class, k)
                {
                    const int byte = bytes[sg], cls = clss[sg], kk = ks[sg];
                    const int len = list_length(sg, cls), base = 2048 * cls;
                    float rv = kNeg;
                    uint32_t ra = 0xFFFFFFFFu;
                    for (int i = ct; i < len; i += 128) {
                        const uint32_t rw = S.rows[base + i];
                        float corr = 0.f;
                        int nn = 0;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int rho = (rw >> (4 * j)) & 7, o = p + 2 * ((byte >> j) & 1);
                            corr += S.A[sg][j][o][rho];
                            const int v = rank_value(o, rho);
                            nn += v * v;
                        }
                        if ((nn >> 4) == kk && (corr > rv || (corr == rv && uint32_t(i) < ra))) {
                            rv = corr;
                            ra = uint32_t(i);
                        }
                    }
                    // reduce within the group of 128 threads (four warps)
#pragma unroll
                    for (int o = 16; o >= 1; o >>= 1) {
                        const float v2 = __shfl_xor_sync(0xFFFFFFFFu, rv, o);
                        const uint32_t a2 = __shfl_xor_sync(0xFFFFFFFFu, ra, o);
                        if (v2 > rv || (v2 == rv && a2 < ra)) {
                            rv = v2;
                            ra = a2;
                        }
                    }
                    __syncthreads();
                    if ((tid & 31) == 0) {
                        S.red_val[tid >> 5] = rv;
                        S.red_arg[tid >> 5] = ra;
                    }
                    __syncthreads();
                    if (ct == 0) {
                        float bv = S.red_val[4 * sg];
                        uint32_t ba = S.red_arg[4 * sg];
                        for (int k = 1; k < 4; ++k) {
                            const float v2 = S.red_val[4 * sg + k];
                            const uint32_t a2 = S.red_arg[4 * sg + k];
                            if (v2 > bv || (v2 == bv && a2 < ba)) {
                                bv = v2;
                                ba = a2;
                            }
                        }
                        S.found_field[sg] = ba == 0xFFFFFFFFu ? 0 : int(ba);
                    }
                    __syncthreads();
                }
                if (tid == 0) {
                    const int n_total = 8 * q + 16 * k3 + norm_residue(p, cls3, bytes[2]);
                    S.best_val = val;
                    S.best_norm = n_total;
                    S.best_corr = val * sqrtf(float(n_total));
                    S.best_path = uint32_t(s8) | (uint32_t(b1) << 6) | (uint32_t(b2) << 7) | (uint32_t(b3) << 11) |
                                  (uint32_t(p) << 12) | (uint32_t(cls1) << 13);
                    S.best_field[0] = S.found_field[0];
                    S.best_field[1] = cls2 ? kMiddleClass0 + S.found_field[1] : S.found_field[1];
                    S.best_field[2] = S.found_field[2];
                }
            }
            __syncthreads();
        }

        if (tid == 0) {
            const uint32_t path = S.best_path;
            const float sg_ = sigma ? sigma[block] : 1.f;
            // gain bit: argmin_g (gain sigma)^2 - 2 gain sigma <w, y> / |y|
            const float c = S.best_val;
            const float e0 = gain0 * sg_ * (gain0 * sg_ - 2.f * c), e1 = gain1 * sg_ * (gain1 * sg_ - 2.f * c);
            const uint64_t gbit = e1 < e0 ? 1u : 0u;
            const uint64_t word = uint64_t(S.best_field[0]) | (uint64_t(S.best_field[1]) << 11) |
                                  (uint64_t(S.best_field[2]) << 22) | (uint64_t(path & 63u) << 33) |
                                  (uint64_t((path >> 6) & 1u) << 39) | (uint64_t((path >> 7) & 15u) << 40) |
                                  (uint64_t((path >> 11) & 1u) << 44) | (uint64_t((path >> 12) & 1u) << 45) |
                                  (uint64_t((path >> 13) & 1u) << 46) | (gbit << 47);
            for (int k = 0; k < 6; ++k) codes[block * 6 + k] = uint8_t(word >> (8 * k));
            if (cosine) cosine[block] = S.best_val / sqrtf(wn2);
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_encode(const float* w, const float* sigma, const void* table, unsigned char* codes, float* cosine,
                          size_t nblocks, cudaStream_t s) {
    int sms = 0;
    cudaError_t e = device_sms(&sms);
    if (e != cudaSuccess) return e;
    const int smem = int(sizeof(EncShared));
    static PerDeviceOnce once;
    e = once.run([smem] { return cudaFuncSetAttribute(k_encode, cudaFuncAttributeMaxDynamicSharedMemorySize, smem); });
    if (e != cudaSuccess) return e;
    const unsigned grid = unsigned(nblocks < size_t(sms) ? nblocks : size_t(sms));
    k_encode<<<grid, kEncThreads, smem, s>>>(w, sigma, static_cast<const DeviceTables*>(table), codes, cosine, nblocks);
    return cudaGetLastError();
}

}  // namespace tetra
