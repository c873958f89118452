// Decode-and-multiply (Eq. (2), Sec. 5.1) for ONE matrix or a short list of
// matrices in a single launch, with no scratch memory: the kernel behind
// tetra_gemv, tetra_gemv_tail and tetra_gemv_list.
//
// Sec. 5.2 of the paper times one launch per matrix; on B200 such a launch holds
// a few microseconds of work, so what is left of it is a chain of latencies.  The
// kernel is arranged to shorten that chain:
//   * everything that does not depend on the activations is started before the
//     kernel waits for its predecessor in the stream (programmatic dependent
//     launch): the decode tables are staged, every warp's first code record is
//     on its way into shared memory, the row scales and tails are pulled into L2;
//   * a CTA of 256 threads takes at most half an SM, so the CTAs of the next
//     launch become resident, and do all of the above, while this launch runs;
//   * after the wait a CTA turns the activations of the matrix it works on into
//     their fixed-point image in shared memory (once per CTA, one column per
//     thread), and its warps split the (row group, column group) passes of the
//     CTA's rows evenly and in memory order, with the decoder, the per-warp
//     cp.async ring and the transpose reduction of the planned-list kernel;
//   * per-(row group, warp) partial sums meet in shared memory and are added in
//     warp order (deterministic), then row scale and tail.
// The only waits are CTA barriers, cp.async.wait_group and griddepcontrol.wait.
#include "../../include/tetra.h"
#include "tetra_gemv_common.cuh"

namespace tetra {

static_assert(kListMax == TETRA_LIST_MAX, "list length limit must agree with the header");

constexpr int kChunkGroups = 32;  // row groups whose partial sums share the shared-memory buffer

struct ListSmem {
    // offsets from the 16 KiB-aligned table copy; total includes the alignment slack
    uint32_t xq, xtail, ring, red, part, rs, tail, total;
};
__host__ __device__ inline ListSmem list_smem(int warps, int image_cols) {
    ListSmem S;
    S.xq = uint32_t(kFastBytes);
    S.xtail = S.xq + uint32_t(image_cols) * kXqBytesPerCol;               // float [24]: x beyond the last word
    S.ring = S.xtail + 96u;
    S.red = S.ring + uint32_t(warps) * 3072u;
    S.part = S.red + uint32_t(warps) * kRedFloats * 4u;
    S.rs = S.part + uint32_t(kChunkGroups * warps * 8 * 4);              // float [chunk rows]: row scales
    S.tail = S.rs + uint32_t(kChunkGroups * 8 * 4);                       // half [chunk rows][24]: tails
    S.total = S.tail + uint32_t(kChunkGroups * 8 * 24 * 2) + kSmAlign;
    return S;
}

__device__ __forceinline__ void ring_fetch(uint32_t dst, const uint4* src, uint32_t Bu) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(src));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst + 512), "l"(src + Bu));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst + 1024), "l"(src + 2 * Bu));
}

// Geometry of one chunk (row groups [ga, ga + ng) of a matrix with Bu words per row).  Its cells
// (row group, column) are numbered row group by row group, Bs = max(Bu, 32) to a row group (cells
// with column >= Bu are empty), and a pass is 32 consecutive cells: no lane idles at the end of a
// row because the next row group's first columns fill the pass.  Warp w of W takes passes
// [passes w / W, passes (w + 1) / W).
struct Chunk {
    uint32_t Bu, Bs;
    int ga, ng, passes;
};
__device__ __forceinline__ Chunk make_chunk(const Problem& P, int ga, int ng) {
    Chunk C;
    C.Bu = uint32_t(P.tail ? P.K / 24 : (P.K + 23) / 24);
    C.Bs = C.Bu < 32u ? 32u : C.Bu;
    C.ga = ga;
    C.ng = ng;
    C.passes = int((uint32_t(ng) * C.Bs + 31u) >> 5);
    return C;
}

// IMAGE: the CTA keeps the fixed-point image of the matrix's activations in shared memory
// (one 80-byte record per column); otherwise (more columns than fit) a lane builds its column's
// record from x for every pass.
template <int THREADS, bool IMAGE>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 2 : 1)
k_gemv_list(const DeviceTables* __restrict__ tab, const __grid_constant__ ListDesc L, int batch) {
    constexpr int W = THREADS / 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pdl_release();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const ListSmem S = list_smem(W, IMAGE ? L.max_blocks : 0);
    unsigned char* smem = stage_fast_tables_async(tab, smem_raw);
    const uint32_t sm_tab = smem_u32(smem);
    float* red = reinterpret_cast<float*>(smem + S.red) + warp * kRedFloats;
    float* part = reinterpret_cast<float*>(smem + S.part);
    float* xtail = reinterpret_cast<float*>(smem + S.xtail);
    float* rs_sm = reinterpret_cast<float*>(smem + S.rs);
    __half* tail_sm = reinterpret_cast<__half*>(smem + S.tail);
    const uint32_t ring = sm_tab + S.ring + uint32_t(warp) * 3072u + uint32_t(lane) * 16u;

    // This CTA's share of the row groups of the whole list, in list order.
    const int g_lo = int((long long)blockIdx.x * L.total_groups / gridDim.x);
    const int g_hi = int((long long)(blockIdx.x + 1) * L.total_groups / gridDim.x);
    if (g_lo >= g_hi) return;
    int p_first = 0;
    while (L.group_prefix[p_first + 1] <= g_lo) ++p_first;

    // Row scales and tails of a chunk's rows into shared memory (they are constants of the model, so
    // this may run before the wait below).  cp.async where the addresses allow it, so that nothing
    // here waits for memory; the caller waits for the group.
    auto stage_rows = [&](const Problem& P, int ga, int ng) {
        const int ntail = P.tail ? P.K % 24 : 0;
        const int rows = min(ng * 8, P.N - ga * 8);
        const float* rs = P.row_scales + size_t(ga) * 8;
        for (int t = threadIdx.x; t < rows; t += THREADS)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" :: "r"(smem_u32(rs_sm + t)), "l"(rs + t));
        const __half* tl = static_cast<const __half*>(P.tail) + size_t(ga) * 8 * ntail;
        if (ntail && (ntail & 1) == 0 && (reinterpret_cast<uintptr_t>(tl) & 3) == 0) {
            const int pairs = ntail >> 1;  // two tail values per 4-byte request
            for (int i = threadIdx.x; i < rows * pairs; i += THREADS) {
                const int t = i / pairs, k = i - t * pairs;
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;"
                             :: "r"(smem_u32(tail_sm + t * 24 + 2 * k)), "l"(tl + size_t(t) * ntail + 2 * k));
            }
        } else {
            for (int i = threadIdx.x; i < rows * ntail; i += THREADS) {
                const int t = i / ntail, k = i - t * ntail;
                tail_sm[t * 24 + k] = tl[size_t(t) * ntail + k];
            }
        }
    };
    // Lane's first cell of pass `ps`: row group (within the chunk) and column.
    auto cell_of = [&](const Chunk& C, int ps, int* rgl, uint32_t* col) {
        const uint32_t cell = uint32_t(ps) * 32u + uint32_t(lane);
        const uint32_t r = cell / C.Bs;
        *rgl = int(r);
        *col = cell - r * C.Bs;
    };
    auto record_ptr = [&](const Problem& P, const Chunk& C, int rgl, uint32_t col) -> const uint4* {
        const int rg = min(rgl, C.ng - 1);
        return static_cast<const uint4*>(P.codes) + size_t(C.ga + rg) * 3 * C.Bu + min(col, C.Bu - 1);
    };

    // ---- before the wait: work that does not depend on the activations ----------------------
    bool first_chunk = true;
    {
        const Problem& P = L.problems[p_first];
        const int ga = g_lo - L.group_prefix[p_first];
        const int ng = min(min(g_hi, L.group_prefix[p_first + 1]) - g_lo, kChunkGroups);
        const Chunk C = make_chunk(P, ga, ng);
        const int ps0 = C.passes * warp / W, ps1 = C.passes * (warp + 1) / W;
        if (ps0 < ps1) {
            int rgl;
            uint32_t col;
            cell_of(C, ps0, &rgl, &col);
            ring_fetch(ring, record_ptr(P, C, rgl, col), C.Bu);
        }
        stage_rows(P, ga, ng);
        asm volatile("cp.async.commit_group;");
    }
    pdl_wait();  // the activations may come from the previous kernel of the stream
    asm volatile("cp.async.wait_group 0;" ::: "memory");  // tables, first rows and first record (the barrier follows)

    int parity = 0;
    for (int job = 0; job < batch; ++job) {  // activation vector `job` of every matrix
        int p = p_first;
        int p_staged = -1;  // matrix whose activations are in the shared-memory image
        for (int g = g_lo; g < g_hi;) {
            while (L.group_prefix[p + 1] <= g) ++p;
            const Problem& P = L.problems[p];
            const int seg_end = min(g_hi, L.group_prefix[p + 1]);
            const int ntail = P.tail ? P.K % 24 : 0;
            const __half* xj = static_cast<const __half*>(P.x) + size_t(job) * P.K;
            float* yj = P.y + size_t(job) * P.N;
            const int ga = g - L.group_prefix[p];
            const int ng = min(seg_end - g, kChunkGroups);
            const Chunk C = make_chunk(P, ga, ng);
            const uint32_t Bu = C.Bu;

            __syncthreads();  // the previous chunk's epilogue has read its buffers; its passes have read the image
            for (int i = threadIdx.x; i < ng * W * 8; i += THREADS) part[i] = 0.f;
            if (!first_chunk) {
                stage_rows(P, ga, ng);
                asm volatile("cp.async.commit_group;");
                asm volatile("cp.async.wait_group 0;" ::: "memory");
            }
            if (p_staged != p) {
                const float xt = (threadIdx.x < 24 && int(threadIdx.x) < ntail) ? __half2float(xj[24 * Bu + threadIdx.x]) : 0.f;
                if (IMAGE) {
                    for (int c = threadIdx.x; c < int(Bu); c += THREADS) {
                        uint32_t q[20];
                        quantise_column(xj, P.K, c, q);
                        uint4* dst = reinterpret_cast<uint4*>(smem + S.xq + c * kXqBytesPerCol);
#pragma unroll
                        for (int k = 0; k < 5; ++k) dst[k] = make_uint4(q[4 * k], q[4 * k + 1], q[4 * k + 2], q[4 * k + 3]);
                    }
                }
                if (threadIdx.x < 24) xtail[threadIdx.x] = xt;
                p_staged = p;
            }
            __syncthreads();

            // ---- this warp's passes --------------------------------------------------------
            const int ps0 = C.passes * warp / W, ps1 = C.passes * (warp + 1) / W;
            if (ps0 < ps1) {
                int rgl;
                uint32_t col;
                cell_of(C, ps0, &rgl, &col);
                if (!first_chunk) {
                    ring_fetch(ring + uint32_t(parity * 1536), record_ptr(P, C, rgl, col), Bu);
                    asm volatile("cp.async.commit_group;");
                }
                int rg_acc = __shfl_sync(0xFFFFFFFFu, rgl, 0);  // row group the accumulators belong to
                float acc[8];
#pragma unroll
                for (int r = 0; r < 8; ++r) acc[r] = 0.f;
                // folds the accumulators of row group rg_acc into this warp's slot of the partial sums
                auto flush = [&]() {
                    float sum = transpose_partial(red, lane, acc);
                    sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
                    sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
                    if ((lane & 3) == 0) part[(rg_acc * W + warp) * 8 + (lane >> 2)] = sum;
                };
                for (int ps = ps0; ps < ps1; ++ps) {
                    uint4 a, b, h;
                    asm volatile("cp.async.wait_group 0;" ::: "memory");
                    {
                        const uint32_t src = ring + uint32_t(parity * 1536);
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "r"(src));
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "r"(src + 512));
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(h.x), "=r"(h.y), "=r"(h.z), "=r"(h.w) : "r"(src + 1024));
                    }
                    // this lane's cell of the next pass: 32 cells on, at most one row group further
                    int nrgl = rgl;
                    uint32_t ncol = col + 32u;
                    if (ncol >= C.Bs) { ncol -= C.Bs; ++nrgl; }
                    if (ps + 1 < ps1) ring_fetch(ring + uint32_t((parity ^ 1) * 1536), record_ptr(P, C, nrgl, ncol), Bu);
                    asm volatile("cp.async.commit_group;");
                    const bool active = rgl < C.ng && col < Bu;
                    LaneX X;
                    {
                        uint32_t q[20];
                        if (IMAGE) {
                            const uint4* src = reinterpret_cast<const uint4*>(smem + S.xq + min(col, Bu - 1) * kXqBytesPerCol);
#pragma unroll
                            for (int k = 0; k < 5; ++k) {
                                const uint4 u = src[k];
                                q[4 * k] = u.x; q[4 * k + 1] = u.y; q[4 * k + 2] = u.z; q[4 * k + 3] = u.w;
                            }
                        } else {
                            quantise_column(xj, P.K, int(min(col, Bu - 1)), q);
                        }
                        lane_x_from_words(q, active, X);
                    }
                    // Lanes of the pass sit in row group rg_acc or, behind a row boundary, in the next one.
                    // The former add to the accumulators; the latter wait until the accumulators have been
                    // folded and then start the next row group's.
                    const int rg_last = __shfl_sync(0xFFFFFFFFu, rgl, 31);
                    if (rg_last == rg_acc) {
                        record_accumulate(sm_tab, a, b, h, X, acc);
                    } else {
                        float v[8];
                        record_values(sm_tab, a, b, h, X, v);
                        const bool mine = rgl == rg_acc;
#pragma unroll
                        for (int r = 0; r < 8; ++r) acc[r] += mine ? v[r] : 0.f;
                        flush();
                        rg_acc = rg_last;
#pragma unroll
                        for (int r = 0; r < 8; ++r) acc[r] = mine ? 0.f : v[r];
                    }
                    parity ^= 1;
                    rgl = nrgl;
                    col = ncol;
                }
                if (rg_acc < C.ng) flush();
            }
            first_chunk = false;
            __syncthreads();
            // ---- epilogue: eight threads per row.  Thread j of a row takes warp j's partial sum (W = 8)
            // or warps j and j + 8 (W = 16) and every eighth tail product; three shuffles add them in a
            // fixed order; row scale, tail (Sec. 5.1), store.
            for (int i = threadIdx.x; i < ng * 64; i += THREADS) {
                const int t = i >> 3, j = i & 7;
                const float* pr = part + (t >> 3) * W * 8 + (t & 7);
                float v = pr[8 * j];
                if (W == 16) v += pr[8 * (j + 8)];
                v *= rs_sm[t];
                for (int k = j; k < ntail; k += 8) v = fmaf(__half2float(tail_sm[t * 24 + k]), xtail[k], v);
                v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
                v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
                v += __shfl_xor_sync(0xFFFFFFFFu, v, 4);
                const int row = ga * 8 + t;
                if (j == 0 && row < P.N) yj[row] = v;
            }
            g += ng;
        }
    }
}


cudaError_t launch_gemv_list(const ListDesc& list, int batch, const void* table, cudaStream_t s) {
    int sms = 0;
    cudaError_t e = device_sms(&sms);
    if (e != cudaSuccess) return e;
    static PerDeviceOnce once;
    e = once.run([] {
        cudaError_t r = cudaFuncSetAttribute(k_gemv_list<256, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (r == cudaSuccess) r = cudaFuncSetAttribute(k_gemv_list<512, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (r == cudaSuccess) r = cudaFuncSetAttribute(k_gemv_list<512, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        return r;
    });
    if (e != cudaSuccess) return e;
    // Two CTAs of eight warps per SM when their shared memory fits side by side (the next launch's
    // CTAs can then start early); one CTA of sixteen warps otherwise; and without the shared-memory
    // image of the activations when even that does not fit.
    const ListSmem small = list_smem(8, list.max_blocks), large = list_smem(16, list.max_blocks);
    const DeviceTables* tab = static_cast<const DeviceTables*>(table);
    if (2u * (small.total + 1024u) <= 227u * 1024u) {
        const int grid = list.total_groups < 2 * sms ? list.total_groups : 2 * sms;
        return launch_pdl(k_gemv_list<256, true>, grid, 256, small.total, s, tab, list, batch);
    }
    const int grid = list.total_groups < sms ? list.total_groups : sms;
    if (large.total <= 227u * 1024u) return launch_pdl(k_gemv_list<512, true>, grid, 512, large.total, s, tab, list, batch);
    return launch_pdl(k_gemv_list<512, false>, grid, 512, list_smem(16, 0).total, s, tab, list, batch);
}

}  // namespace tetra
