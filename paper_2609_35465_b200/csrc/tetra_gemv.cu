// Decode-and-multiply kernels (Eq. (2), Sec. 5.1) for sm_100a.
//
//   k_gemv_paper  the thread layout the paper describes for its own GPU: a warp
//                 per output row, a lane per block, the six table loads of
//                 Fig. "decode", FP32 multiply-accumulate, shuffle reduction.
//                 Kept as a comparison arm and cross-check.
//   k_gemv_units  the B200 design (also in k_gemv_list, tetra_list.cu): a lane owns one block column and keeps its
//                 24 activations in registers as 24-bit fixed point (three int8
//                 planes, power-of-two step per block column, so float16 inputs
//                 within 2^12 of the column's largest are held exactly); it
//                 walks the rows, decodes each word into packed int8 with PRMT
//                 lookups and multiplies with DP4A: products and the sum over
//                 a block are exact integers, one rounding when the block's sum
//                 becomes a float, FP32 accumulation across blocks.  The ALU
//                 pipe only unpacks fields; the integer-MAD pipe does the
//                 arithmetic.
//                 k_gemv_units serves a planned list of matrices from one
//                 persistent grid: k_prepare_x first writes the fixed-point
//                 activations of every matrix to the plan's scratch area, then
//                 every warp walks independent units (eight rows of one matrix,
//                 all columns), so no warp ever waits for another.
#include <cuda_fp16.h>

#include <cstdlib>
#include <cstring>
#include <mutex>

#include "tetra_gemv_common.cuh"

namespace tetra {

cudaError_t device_sms(int* sms) {
    static std::mutex mu;
    static int cached[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == 0) {
        int n = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        cached[dev] = n;
    }
    *sms = cached[dev];
    return cudaSuccess;
}

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
// Planned list of matrices: k_prepare_x + k_gemv_units
// ===========================================================================
// Workspace written by grouped_plan (host) and read by both kernels:
//   PlanHeader | Problem[count] | unit_prefix[count + 1] | col_prefix[count + 1]
//              | warp_start[nwarps + 1] (optional) | pad | xq records
// A unit is groups_per_unit(B) consecutive row groups of one matrix, all columns.
struct PlanHeader {
    int32_t count;
    int32_t total_units;  // sum over matrices of their units
    int32_t total_cols;   // sum over matrices of words per row
    int32_t nwarps;       // warps the unit ranges were cut for (0: no ranges, units are dealt round-robin)
    uint32_t off_problems, off_unit_prefix, off_col_prefix, off_xq;
    uint32_t off_warp_start;
    // fine mode (small lists): a unit is one row group x a slice of the column groups
    uint32_t off_fine;      // FineInfo[count], 0 in coarse mode
    uint32_t off_counters;  // int32 per row group: slices of the group that have finished
    uint32_t off_partials;  // float [row group][slice][8]
    int32_t total_groups;
    // coarse mode with unit ranges: units [0, dyn_start) are cut into the warps' ranges; the units from
    // dyn_start on are claimed one at a time through dyn_next by warps that have finished their range
    // (k_prepare_x sets dyn_next = dyn_start before every run)
    int32_t dyn_start;
    int32_t dyn_next;
    int32_t pad_[1];
};
#ifndef TETRA_DYN_PERMILLE
#define TETRA_DYN_PERMILLE 100
#endif
constexpr int kDynamicTailPermille = TETRA_DYN_PERMILLE;  // share of the list's work left for the claimed units

struct FineInfo {
    int32_t slices;          // column slices per row group
    int32_t cgs_per_slice;   // column groups per slice (the last slice may hold fewer)
    int32_t group_prefix;    // row groups of the matrices before this one
    int32_t partial_prefix;  // floats of partial sums before this matrix
};

constexpr int kMaxPlanWarps = 8192;    // room reserved for warp_start in a planned list's workspace
constexpr long long kFineMaxTasks = 65536;  // upper bound of the (row group, column group) pairs of a fine-mode list

static inline long long problem_tasks(const Problem& q);

static size_t plan_meta_bytes(int count, int nwarps) {
    size_t b = sizeof(PlanHeader) + size_t(count) * sizeof(Problem) + 2 * size_t(count + 1) * 4 +
               (nwarps ? size_t(nwarps + 1) * 4 : 0) + size_t(count) * sizeof(FineInfo);
    return (b + 255) & ~size_t(255);
}

static inline int problem_blocks(const Problem& q) {
    return (q.tail || q.K % 24 == 0) ? q.K / 24 : (q.K + 23) / 24;
}

// Row groups (of eight rows) one unit covers.  When the last column group of a matrix is at most
// half full (B mod 32 in 1..16), up to three consecutive row groups share one pass over it, so that
// pass runs with most lanes busy instead of B mod 32 of them.
__host__ __device__ inline int groups_per_unit(int B) {
    const int rem = B & 31;
    if (rem == 0 || rem > 16) return 1;
    const int r = 32 / rem;
    return r < 3 ? r : 3;
}
static inline long long problem_tasks(const Problem& q) {
    return (long long)((q.N + 7) / 8) * ((problem_blocks(q) + 31) / 32);
}
// Space for the fine mode is reserved for every list of at most kFineMaxTasks (row group, column group)
// pairs; the plan then takes the fine mode when the list has at most five such pairs per warp of the
// grid (measured on B200: below that the coarse units leave most warps idle, above it the fine mode's
// partial sums and counters cost more than they gain).
static bool list_may_be_fine(const Problem* problems, int count) {
    long long tasks = 0;
    for (int i = 0; i < count; ++i) tasks += problem_tasks(problems[i]);
    return tasks <= kFineMaxTasks;
}
static bool list_is_fine(const Problem* problems, int count, int nwarps) {
    long long tasks = 0;
    for (int i = 0; i < count; ++i) tasks += problem_tasks(problems[i]);
    return tasks <= kFineMaxTasks && tasks <= 5LL * (nwarps ? nwarps : 2048);
}
static inline int problem_units(const Problem& q) {
    const int R = groups_per_unit(problem_blocks(q));
    return ((q.N + 7) / 8 + R - 1) / R;
}

size_t grouped_workspace_bytes(const Problem* problems, int count) {
    size_t cols = 0;
    for (int i = 0; i < count; ++i) cols += size_t(problem_blocks(problems[i]));
    size_t bytes = plan_meta_bytes(count, kMaxPlanWarps) + cols * kXqBytesPerCol;
    if (list_may_be_fine(problems, count)) {  // counters and partial sums of the fine mode
        long long groups = 0, tasks = 0;
        for (int i = 0; i < count; ++i) { groups += (problems[i].N + 7) / 8; tasks += problem_tasks(problems[i]); }
        bytes = ((bytes + 255) & ~size_t(255)) + size_t(groups) * 4 + 256 + size_t(tasks) * 8 * 4;
    }
    return bytes;
}

// Largest p with prefix[p] <= v (prefix[0] = 0, prefix[count] > v).
__device__ __forceinline__ int find_problem(const int32_t* __restrict__ prefix, int count, int v) {
    int lo = 0, hi = count;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(prefix + mid) <= v) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(256) k_prepare_x(unsigned char* __restrict__ ws) {
    pdl_release();
    pdl_wait();  // the activations (and the plan) may come from the previous kernel of the stream
    const PlanHeader* H = reinterpret_cast<const PlanHeader*>(ws);
    const Problem* problems = reinterpret_cast<const Problem*>(ws + H->off_problems);
    const int32_t* col_prefix = reinterpret_cast<const int32_t*>(ws + H->off_col_prefix);
    uint4* xq = reinterpret_cast<uint4*>(ws + H->off_xq);
    for (int gc = blockIdx.x * blockDim.x + threadIdx.x; gc < H->total_cols; gc += gridDim.x * blockDim.x) {
        const int p = find_problem(col_prefix, H->count, gc);
        const Problem P = problems[p];
        uint32_t q[20];
        quantise_column(static_cast<const __half*>(P.x), P.K, gc - col_prefix[p], q);
#pragma unroll
        for (int k = 0; k < 5; ++k) xq[size_t(gc) * 5 + k] = make_uint4(q[4 * k], q[4 * k + 1], q[4 * k + 2], q[4 * k + 3]);
    }
    if (!H->off_fine && blockIdx.x == 0 && threadIdx.x == 0)
        reinterpret_cast<PlanHeader*>(ws)->dyn_next = H->dyn_start;  // the claimed units start over
    if (H->off_fine) {  // fine mode: the per-row-group arrival counters start every run at zero
        int32_t* counters = reinterpret_cast<int32_t*>(ws + H->off_counters);
        for (int g = blockIdx.x * blockDim.x + threadIdx.x; g < H->total_groups; g += gridDim.x * blockDim.x)
            counters[g] = 0;
    }
}

// This lane's activation record (global memory, L1/L2 resident) into registers.
__device__ __forceinline__ void load_lane_x(const unsigned char* xq_rec, bool active, LaneX& X) {
    const uint4* src = reinterpret_cast<const uint4*>(xq_rec);
    const uint4 t0 = __ldg(src), t1 = __ldg(src + 1), t2 = __ldg(src + 2), t3 = __ldg(src + 3), t4 = __ldg(src + 4);
    X.hi[0] = t0.x; X.hi[1] = t0.y; X.hi[2] = t0.z; X.hi[3] = t0.w; X.hi[4] = t1.x; X.hi[5] = t1.y;
    X.mid[0] = t1.z; X.mid[1] = t1.w; X.mid[2] = t2.x; X.mid[3] = t2.y; X.mid[4] = t2.z; X.mid[5] = t2.w;
    X.lo[0] = t3.x; X.lo[1] = t3.y; X.lo[2] = t3.z; X.lo[3] = t3.w; X.lo[4] = t4.x; X.lo[5] = t4.y;
    X.step = active ? __uint_as_float(t4.z) : 0.f;  // an inactive lane contributes exact zeros
    X.sum = int(t4.w);
}

#ifndef TETRA_UNIT_THREADS
#define TETRA_UNIT_THREADS 512
#endif
constexpr int kUnitThreads = TETRA_UNIT_THREADS;
constexpr int kUnitWarps = kUnitThreads / 32;

// Coarse mode: every warp walks its range of units (up to three row groups of one matrix, all columns).
__device__ __forceinline__ void units_coarse(unsigned char* __restrict__ ws, unsigned char* smem, uint32_t sm_tab) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* red = reinterpret_cast<float*>(smem + kFastBytes) + warp * kRedFloats;
    const PlanHeader* H = reinterpret_cast<const PlanHeader*>(ws);
    const Problem* problems = reinterpret_cast<const Problem*>(ws + H->off_problems);
    const int32_t* unit_prefix = reinterpret_cast<const int32_t*>(ws + H->off_unit_prefix);
    const int32_t* col_prefix = reinterpret_cast<const int32_t*>(ws + H->off_col_prefix);
    const unsigned char* xq_all = ws + H->off_xq;
    const int total_units = H->total_units;

    // Units of this warp: a contiguous range cut for equal work when the plan holds ranges for this
    // grid (neighbouring warps then walk neighbouring row groups of the same matrices), else every
    // (warps in grid)-th unit.
    const int gw = blockIdx.x * kUnitWarps + warp, nw = gridDim.x * kUnitWarps;
    int u = gw, u_end = total_units, u_step = nw;
    bool claim = false;  // after the range: claim the units from dyn_start on, one at a time
    if (H->nwarps == nw) {
        const int32_t* warp_start = reinterpret_cast<const int32_t*>(ws + H->off_warp_start);
        u = __ldg(warp_start + gw);
        u_end = __ldg(warp_start + gw + 1);
        u_step = 1;
        claim = H->dyn_start < total_units;
    }
    int p = -1, p_begin = 0, p_end = 0;  // matrix of the current unit and its range of units
    // per matrix, kept in registers across its units (everything else is re-read where it is needed)
    const uint4* codes_p = nullptr;
    const unsigned char* xq_p = xq_all;
    int G = 1;
    uint32_t Bu = 1;
    bool have_record = false;            // the ring already holds the first record of the unit about to start
    // Code records reach the decoder through a per-warp ring in shared memory: two slots of 3 x 512
    // bytes (one 16-byte part per lane), filled with cp.async one pass ahead, so the prefetch holds
    // no registers while eight blocks are being decoded.  Each lane reads back only what it copied.
    const uint32_t ring = sm_tab + uint32_t(kFastBytes) + uint32_t(kUnitWarps * kRedFloats * 4) + uint32_t(warp) * 3072u + uint32_t(lane) * 16u;
    int pass_parity = 0;

    for (;; u += u_step) {
        if (u >= u_end) {
            if (!claim) break;
            // The range is done: claim one of the units that were left unassigned.  One atomic per unit; it
            // only hands out numbers, nothing waits on it, and the numbers a warp gets increase, so the walk
            // below still only goes up.  (Claiming one unit ahead would hide the atomic's latency but keeps a
            // register live across the passes, which costs more than it saves.)
            int c = 0;
            if (lane == 0) c = atomicAdd(&reinterpret_cast<PlanHeader*>(ws)->dyn_next, 1);
            c = __shfl_sync(0xFFFFFFFFu, c, 0);
            if (c >= total_units) break;
            u = c;
            u_end = c + 1;
            have_record = false;
        }
        if (u >= p_end) {  // first unit, or the walk has left the matrix: units only go up
            do { ++p; p_end = __ldg(unit_prefix + p + 1); } while (u >= p_end);
            p_begin = __ldg(unit_prefix + p);
            const Problem& Q = problems[p];
            const int K = Q.K;
            Bu = uint32_t(Q.tail ? K / 24 : (K + 23) / 24);
            G = (Q.N + 7) / 8;
            codes_p = static_cast<const uint4*>(Q.codes);
            xq_p = xq_all + size_t(__ldg(col_prefix + p)) * kXqBytesPerCol;
            have_record = false;
        }
        const int CGf = int(Bu >> 5);   // full column groups
        const int rem = int(Bu & 31);   // columns of the last, partial one
        const int R = groups_per_unit(int(Bu));
        const int g0 = (u - p_begin) * R;
        const int ng = min(R, G - g0);
        const uint4* codes0 = codes_p + size_t(g0) * 3 * Bu;
        // this lane's place in the joint pass over the partial column group: row group, column
        const int lane_grp = rem ? min(lane / max(rem, 1), 3) : 0;
        const bool lane_in = rem && lane_grp < ng;
        const uint32_t lane_col = uint32_t(CGf * 32) + (lane_in ? uint32_t(lane - lane_grp * rem) : 0u);
        const uint4* rem_rec = codes0 + size_t(lane_in ? lane_grp : 0) * 3 * Bu + lane_col;
        const bool next_unit_here = CGf > 0 && u + u_step < min(u_end, p_end);

        if (!have_record) {
            const uint4* first = CGf > 0 ? codes0 + lane : rem_rec;
            const uint32_t dst = ring + uint32_t(pass_parity * 1536);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(first));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst + 512), "l"(first + Bu));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst + 1024), "l"(first + 2 * Bu));
            asm volatile("cp.async.commit_group;");
        }
        have_record = false;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f;  // per row group: this lane's partial row sum (row lane / 4)
        float acc[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) acc[r] = 0.f;

        // One pass = one 48-byte record per lane: the full column groups of each row group in turn,
        // then the joint pass over the partial column group (a single call site of the decoder).
        const int full_passes = ng * CGf, passes = full_passes + (rem ? 1 : 0);
        int gi = 0, cg = 0;
        for (int pass = 0; pass < passes; ++pass) {
            const bool joint = pass >= full_passes;
            uint4 a, b, h;
            {
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                const uint32_t src = ring + uint32_t(pass_parity * 1536);
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "r"(src));
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "r"(src + 512));
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(h.x), "=r"(h.y), "=r"(h.z), "=r"(h.w) : "r"(src + 1024));
            }
            // prefetch the next pass's record (or the first one of this warp's next unit)
            const uint4* next = nullptr;
            if (pass + 1 < full_passes) {
                const bool wrap = cg + 1 == CGf;
                next = codes0 + size_t(wrap ? gi + 1 : gi) * 3 * Bu + (wrap ? 0 : cg + 1) * 32 + lane;
            } else if (pass + 1 < passes) {
                next = rem_rec;
            } else if (next_unit_here) {
                next = codes0 + size_t(u_step) * R * 3 * Bu + lane;
                have_record = true;
            }
            if (next) {
                const uint32_t dst = ring + uint32_t((pass_parity ^ 1) * 1536);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(next));
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst + 512), "l"(next + Bu));
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst + 1024), "l"(next + 2 * Bu));
            }
            asm volatile("cp.async.commit_group;");
            LaneX X;
            load_lane_x(xq_p + (joint ? lane_col : uint32_t(cg * 32 + lane)) * uint32_t(kXqBytesPerCol),
                        !joint || lane_in, X);
            record_accumulate(sm_tab, a, b, h, X, acc);  // acc is zero when the joint pass begins
            pass_parity ^= 1;
            if (!joint) {
                if (++cg == CGf) {  // row group done: fold its eight accumulators into this lane's row
                    const float t = transpose_partial(red, lane, acc);
                    if (gi == 0) s0 = t; else if (gi == 1) s1 = t; else s2 = t;
#pragma unroll
                    for (int r = 0; r < 8; ++r) acc[r] = 0.f;
                    cg = 0;
                    ++gi;
                }
            } else {
                // lane -> (row group, column); lane l then sums, for row l / 4, the columns
                // k = l % 4, l % 4 + 4, ... of every row group's segment of the buffer
                __syncwarp();
#pragma unroll
                for (int r = 0; r < 8; ++r) red[r * kRedStride + lane] = acc[r];
                __syncwarp();
                const float* rr = red + (lane >> 2) * kRedStride;
                for (int k = lane & 3; k < rem; k += 4) {
                    s0 += rr[k];
                    if (R > 1) s1 += rr[rem + k];
                    if (R > 2) s2 += rr[2 * rem + k];
                }
            }
        }
        // row scale, tail (Sec. 5.1; four lanes per row share the tail), store
        {
            const Problem P = problems[p];
            const int ntail = P.tail ? P.K % 24 : 0;
            const __half* xh = static_cast<const __half*>(P.x) + 24 * Bu;
            for (int gk = 0; gk < ng; ++gk) {
                const int row = (g0 + gk) * 8 + (lane >> 2);
                float sum = gk == 0 ? s0 : (gk == 1 ? s1 : s2);
                if (row < P.N) {
                    sum *= __ldg(P.row_scales + row);
                    const __half* tl = static_cast<const __half*>(P.tail) + size_t(row) * ntail;
                    for (int k = lane & 3; k < ntail; k += 4)
                        sum = fmaf(__half2float(tl[k]), __half2float(xh[k]), sum);
                }
                sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
                sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
                if (row < P.N && (lane & 3) == 0) P.y[row] = sum;
            }
        }
    }
}

// Fine mode of the planned list, for lists too small to fill the GPU with coarse units (single
// matrices, the matrices of one layer): a unit is one row group x a slice of the column groups.
// Each unit leaves eight partial row sums in the scratch area and bumps its row group's counter; the
// unit that finds all the other slices done adds them up in slice order (fixed order, no waiting,
// no floating-point atomics), applies the row scale and the tail, and stores.
__device__ __noinline__ void units_fine(unsigned char* __restrict__ ws, unsigned char* smem, uint32_t sm_tab) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* red = reinterpret_cast<float*>(smem + kFastBytes) + warp * kRedFloats;
    const PlanHeader* H = reinterpret_cast<const PlanHeader*>(ws);
    const Problem* problems = reinterpret_cast<const Problem*>(ws + H->off_problems);
    const int32_t* unit_prefix = reinterpret_cast<const int32_t*>(ws + H->off_unit_prefix);
    const int32_t* col_prefix = reinterpret_cast<const int32_t*>(ws + H->off_col_prefix);
    const FineInfo* fine = reinterpret_cast<const FineInfo*>(ws + H->off_fine);
    int32_t* counters = reinterpret_cast<int32_t*>(ws + H->off_counters);
    float* partials = reinterpret_cast<float*>(ws + H->off_partials);
    const unsigned char* xq_all = ws + H->off_xq;
    const int total_units = H->total_units;
    const uint32_t ring = sm_tab + uint32_t(kFastBytes) + uint32_t(kUnitWarps * kRedFloats * 4) +
                          uint32_t(warp) * 3072u + uint32_t(lane) * 16u;

    // equal shares of consecutive units per warp (units of a list in fine mode are of similar size)
    const int gw = blockIdx.x * kUnitWarps + warp, nw = gridDim.x * kUnitWarps;
    int u = int((long long)total_units * gw / nw);
    const int u_end = int((long long)total_units * (gw + 1) / nw);
    int p = -1, p_begin = 0, p_end = 0;
    Problem P{};
    FineInfo F{};
    int CG = 1;
    uint32_t Bu = 1;
    const unsigned char* xq_p = xq_all;

    for (; u < u_end; ++u) {
        if (u >= p_end) {
            do { ++p; p_end = __ldg(unit_prefix + p + 1); } while (u >= p_end);
            p_begin = __ldg(unit_prefix + p);
            P = problems[p];
            F = fine[p];
            Bu = uint32_t(P.tail ? P.K / 24 : (P.K + 23) / 24);
            CG = int((Bu + 31) >> 5);
            xq_p = xq_all + size_t(__ldg(col_prefix + p)) * kXqBytesPerCol;
        }
        const int local = u - p_begin;
        const int g = local / F.slices, slice = local - g * F.slices;
        const int c0 = slice * F.cgs_per_slice, c1 = min(CG, c0 + F.cgs_per_slice);
        const uint4* codes = static_cast<const uint4*>(P.codes) + size_t(g) * 3 * Bu;

        float acc[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) acc[r] = 0.f;
        {   // first record of the unit into ring slot 0
            const uint4* first = codes + min(uint32_t(c0 * 32 + lane), Bu - 1);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(ring), "l"(first));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(ring + 512), "l"(first + Bu));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(ring + 1024), "l"(first + 2 * Bu));
            asm volatile("cp.async.commit_group;");
        }
        int parity = 0;
        for (int cg = c0; cg < c1; ++cg) {
            uint4 a, b, h;
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            {
                const uint32_t src = ring + uint32_t(parity * 1536);
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "r"(src));
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "r"(src + 512));
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(h.x), "=r"(h.y), "=r"(h.z), "=r"(h.w) : "r"(src + 1024));
            }
            if (cg + 1 < c1) {
                const uint4* next = codes + min(uint32_t((cg + 1) * 32 + lane), Bu - 1);
                const uint32_t dst = ring + uint32_t((parity ^ 1) * 1536);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(next));
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst + 512), "l"(next + Bu));
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst + 1024), "l"(next + 2 * Bu));
            }
            asm volatile("cp.async.commit_group;");
            const uint32_t col = uint32_t(cg * 32 + lane);
            LaneX X;
            load_lane_x(xq_p + min(col, Bu - 1) * uint32_t(kXqBytesPerCol), col < Bu, X);
            float v[8];
            record_values(sm_tab, a, b, h, X, v);
#pragma unroll
            for (int r = 0; r < 8; ++r) acc[r] += v[r];
            parity ^= 1;
        }
        float sum = transpose_partial(red, lane, acc);
        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
        float* mine = partials + F.partial_prefix + (size_t(g) * F.slices + slice) * 8;
        if ((lane & 3) == 0) mine[lane >> 2] = sum;
        __threadfence();   // the partial sums are visible before the counter moves
        __syncwarp();
        int arrived = 0;
        if (lane == 0) arrived = atomicAdd(counters + F.group_prefix + g, 1);
        arrived = __shfl_sync(0xFFFFFFFFu, arrived, 0);
        if (arrived == F.slices - 1) {  // every slice of this row group is in: finish the rows
            __threadfence();
            const int row = g * 8 + lane;
            if (lane < 8 && row < P.N) {
                const float* all = partials + F.partial_prefix + size_t(g) * F.slices * 8 + lane;
                float total = 0.f;
                for (int k = 0; k < F.slices; ++k) total += __ldcg(all + 8 * k);
                float res = __ldg(P.row_scales + row) * total;
                const int ntail = P.tail ? P.K % 24 : 0;
                const __half* xh = static_cast<const __half*>(P.x) + 24 * Bu;
                const __half* tl = static_cast<const __half*>(P.tail) + size_t(row) * ntail;
                for (int k = 0; k < ntail; ++k) res = fmaf(__half2float(tl[k]), __half2float(xh[k]), res);
                P.y[row] = res;
            }
        }
    }
}

// The persistent kernel of a planned list.  The plan in the workspace says which of the two modes it
// was cut for (PlanHeader::off_fine), so a workspace can be copied or moved and still runs correctly:
// the host needs no record of it.
__global__ void __launch_bounds__(kUnitThreads, 1)
k_gemv_units(const DeviceTables* __restrict__ tab, unsigned char* __restrict__ ws) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pdl_release();
    unsigned char* smem = stage_fast_tables(tab, smem_raw);
    const uint32_t sm_tab = smem_u32(smem);
    __syncthreads();  // the only CTA-wide barrier: tables are staged
    pdl_wait();       // the plan's activation records (and zeroed counters) come from k_prepare_x
    if (reinterpret_cast<const PlanHeader*>(ws)->off_fine) units_fine(ws, smem, sm_tab);
    else units_coarse(ws, smem, sm_tab);
}


cudaError_t grouped_plan(const Problem* problems_host, int count, void* ws_dev, size_t ws_bytes, cudaStream_t s) {
    if (ws_bytes < grouped_workspace_bytes(problems_host, count)) return cudaErrorInvalidValue;
    int sms = 0;
    cudaError_t e = device_sms(&sms);
    if (e != cudaSuccess) return e;
    int nwarps = sms * kUnitWarps;  // the grid grouped_run launches on this device
    if (nwarps > kMaxPlanWarps) nwarps = 0;
    const size_t meta = plan_meta_bytes(count, nwarps);
    unsigned char* buf = static_cast<unsigned char*>(calloc(1, meta));
    if (!buf) return cudaErrorMemoryAllocation;
    PlanHeader* H = reinterpret_cast<PlanHeader*>(buf);
    H->count = count;
    H->nwarps = nwarps;
    H->off_problems = uint32_t(sizeof(PlanHeader));
    H->off_unit_prefix = H->off_problems + uint32_t(count) * uint32_t(sizeof(Problem));
    H->off_col_prefix = H->off_unit_prefix + uint32_t(count + 1) * 4u;
    H->off_warp_start = H->off_col_prefix + uint32_t(count + 1) * 4u;
    H->off_xq = uint32_t(plan_meta_bytes(count, kMaxPlanWarps));
    memcpy(buf + H->off_problems, problems_host, size_t(count) * sizeof(Problem));
    int32_t* up = reinterpret_cast<int32_t*>(buf + H->off_unit_prefix);
    int32_t* cp = reinterpret_cast<int32_t*>(buf + H->off_col_prefix);
    const bool fine_mode = list_is_fine(problems_host, count, nwarps);
    long long units = 0, cols = 0;
    if (fine_mode) {
        // column groups per unit: aim at about four units per warp of the grid
        long long tasks = 0, groups = 0;
        for (int i = 0; i < count; ++i) { tasks += problem_tasks(problems_host[i]); groups += (problems_host[i].N + 7) / 8; }
        const long long want = 4LL * (nwarps ? nwarps : 2048);
        long long per = tasks / want;
        if (per < 1) per = 1;
        H->off_fine = H->off_col_prefix + uint32_t(count + 1) * 4u + (nwarps ? uint32_t(nwarps + 1) * 4u : 0u);
        FineInfo* fi = reinterpret_cast<FineInfo*>(buf + H->off_fine);
        size_t xq_end = size_t(H->off_xq);
        for (int i = 0; i < count; ++i) xq_end += size_t(problem_blocks(problems_host[i])) * kXqBytesPerCol;
        xq_end = (xq_end + 255) & ~size_t(255);
        H->off_counters = uint32_t(xq_end);
        H->off_partials = uint32_t((xq_end + size_t(groups) * 4 + 255) & ~size_t(255));
        H->total_groups = int32_t(groups);
        long long gp = 0, pp = 0;
        for (int i = 0; i < count; ++i) {
            const int CGi = (problem_blocks(problems_host[i]) + 31) / 32, Gi = (problems_host[i].N + 7) / 8;
            const int cps = int(per < CGi ? per : CGi);
            const int slices = (CGi + cps - 1) / cps;
            fi[i] = FineInfo{slices, cps, int32_t(gp), int32_t(pp)};
            up[i] = int32_t(units);
            cp[i] = int32_t(cols);
            units += (long long)Gi * slices;
            cols += problem_blocks(problems_host[i]);
            gp += Gi;
            pp += (long long)Gi * slices * 8;
        }
        nwarps = 0;  // the fine kernel cuts equal shares itself
        H->nwarps = 0;
    } else
    for (int i = 0; i < count; ++i) {
        up[i] = int32_t(units);
        cp[i] = int32_t(cols);
        units += problem_units(problems_host[i]);
        cols += problem_blocks(problems_host[i]);
    }
    up[count] = int32_t(units);
    cp[count] = int32_t(cols);
    if (units > 0x7FFFFFF0LL || cols > 0x7FFFFFF0LL) e = cudaErrorInvalidValue;
    H->total_units = int32_t(units);
    H->total_cols = int32_t(cols);
    if (e == cudaSuccess && nwarps) {
        // Cut the unit sequence into nwarps contiguous ranges of equal work; a unit costs its number of
        // column groups plus a little for its prologue and epilogue.
        auto unit_work = [&](int i) {
            const int Bi = problem_blocks(problems_host[i]);
            return (long long)(groups_per_unit(Bi) * (Bi / 32) + (Bi % 32 ? 1 : 0)) * 8 + 2;
        };
        long long total = 0;
        for (int i = 0; i < count; ++i) total += unit_work(i) * problem_units(problems_host[i]);
        // The last tenth of the work is not assigned: warps that finish early claim it unit by unit, which
        // evens out what the cost model and the SMs' unequal speeds leave (measured on the Qwen3-8B pass:
        // the average scheduler idled 4.2 % of the kernel's time behind the slowest one).  Only when a warp
        // has at least a few units.
        H->dyn_start = int32_t(units);
        if (units >= 8LL * nwarps) {
            const long long planned = total - total * kDynamicTailPermille / 1000;
            long long acc = 0;
            int i = 0;
            while (i < count - 1 && acc + unit_work(i) * problem_units(problems_host[i]) <= planned) {
                acc += unit_work(i) * problem_units(problems_host[i]);
                ++i;
            }
            long long ds = up[i] + (planned - acc) / unit_work(i);
            if (ds > units) ds = units;
            H->dyn_start = int32_t(ds);
            total = acc + (ds - up[i]) * unit_work(i);
        }
        int32_t* wsx = reinterpret_cast<int32_t*>(buf + H->off_warp_start);
        int pi = 0;
        long long before = 0;  // work of matrices 0..pi-1
        for (int w = 0; w < nwarps; ++w) {
            const long long target = total * w / nwarps;
            while (pi < count - 1 && before + unit_work(pi) * problem_units(problems_host[pi]) <= target) {
                before += unit_work(pi) * problem_units(problems_host[pi]);
                ++pi;
            }
            long long uu = up[pi] + (target - before) / unit_work(pi);
            if (uu > H->dyn_start) uu = H->dyn_start;
            wsx[w] = int32_t(uu);
        }
        wsx[nwarps] = H->dyn_start;
    }
    // pageable source: the runtime stages it before returning, so the buffer can be freed
    if (e == cudaSuccess) e = cudaMemcpyAsync(ws_dev, buf, meta, cudaMemcpyHostToDevice, s);
    free(buf);
    return e;
}

size_t single_plan_meta_bytes() { return plan_meta_bytes(1, 0); }

size_t single_plan_scratch_bytes(int blocks_per_row) {
    return plan_meta_bytes(1, 0) + size_t(blocks_per_row) * kXqBytesPerCol;
}

void single_plan_fill(const Problem& problem, unsigned char* meta_host) {
    memset(meta_host, 0, plan_meta_bytes(1, 0));
    PlanHeader* H = reinterpret_cast<PlanHeader*>(meta_host);
    H->count = 1;
    H->total_units = problem_units(problem);
    H->total_cols = problem_blocks(problem);
    H->off_problems = uint32_t(sizeof(PlanHeader));
    H->nwarps = 0;  // no unit ranges: the kernel deals units round-robin
    H->off_unit_prefix = H->off_problems + uint32_t(sizeof(Problem));
    H->off_col_prefix = H->off_unit_prefix + 8u;
    H->off_xq = uint32_t(plan_meta_bytes(1, 0));
    memcpy(meta_host + H->off_problems, &problem, sizeof(Problem));
    int32_t* up = reinterpret_cast<int32_t*>(meta_host + H->off_unit_prefix);
    int32_t* cp = reinterpret_cast<int32_t*>(meta_host + H->off_col_prefix);
    up[0] = 0; up[1] = H->total_units;
    cp[0] = 0; cp[1] = H->total_cols;
}

cudaError_t grouped_run(void* ws_dev, const void* table, cudaStream_t s) {
    int sms = 0;
    cudaError_t e = device_sms(&sms);
    if (e != cudaSuccess) return e;
    const uint32_t smem = kTableSmemBytes + kUnitWarps * kRedFloats * 4 + kUnitWarps * 3072;
    static PerDeviceOnce once;
    e = once.run([smem] { return cudaFuncSetAttribute(k_gemv_units, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)); });
    if (e != cudaSuccess) return e;
    e = launch_pdl(k_prepare_x, sms * 2, 256, 0, s, static_cast<unsigned char*>(ws_dev));
    if (e != cudaSuccess) return e;
    return launch_pdl(k_gemv_units, sms, kUnitThreads, smem, s, static_cast<const DeviceTables*>(table),
                      static_cast<unsigned char*>(ws_dev));
}

}  // namespace tetra
