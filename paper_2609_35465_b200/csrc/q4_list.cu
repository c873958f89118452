// Batch-1 products of a LIST of 4-bit group-quantised matrices (the int4 projections of a token pass,
// Sec. 4.1, 4.3, 5.1) from one persistent grid.
//
// A single tetra_q4_gemv launch on a projection-sized matrix (2-27 MB) is over in a few microseconds,
// most of them fixed cost: the launch, the per-CTA prologue (group sums of the activations behind a
// barrier), the ring filling up, the pieces combined behind another barrier.  Here the chunks of all
// matrices form one sequence in memory order; every warp of a persistent grid owns a contiguous
// range of it and streams it through its cp.async ring without ever draining it between matrices,
// and no warp waits for another:
//   k_q4_list_prepare  per group of every matrix: sum of x and minus the sum of bias_k x_k (the MMA
//                      operands carry biases 1024 and 64), into the workspace;
//   k_q4_list_main     the stream: dequantise with five logic operations per four registers, MMA
//                      against the activations (read through L1), scale and offset per group;
//                      a strip (32 rows) that lies wholly inside a warp's range is stored, one cut by
//                      a range boundary leaves a piece in the workspace;
//   k_q4_list_combine  adds the pieces of a strip in warp order and stores it.
// Deterministic (fixed order everywhere), no atomics, no waits besides cp.async.wait_group and
// griddepcontrol.wait.
#include <cstdlib>
#include <cstring>

#include "../../include/tetra.h"
#include "../../include/tetra_q4.h"
#include "q4_common.cuh"
#include "tetra_gemv_common.cuh"

namespace tetra {
namespace {

constexpr int kQ4ListThreads = 512;
constexpr int kQ4ListWarps = kQ4ListThreads / 32;
constexpr int kPieceFloats = 32;  // a partial strip: column 0 of its 32 rows (the list call has one vector per matrix)

struct Q4Item {
    const unsigned char* packed;
    const __half* x;
    float* y;
    int32_t N, K;
    int32_t groups, strips;
    uint32_t chunk_begin;  // chunks of the matrices before this one
    uint32_t group_begin;  // groups of the matrices before this one (index into the group sums)
    uint32_t strip_begin;  // strips of the matrices before this one
    uint32_t pad_;
};
static_assert(sizeof(Q4Item) == 56, "descriptor layout");

struct Q4ListHeader {
    int32_t count, G, nwarps, pad0_;
    uint32_t total_chunks, total_groups, total_strips, pad1_;
    uint32_t off_items, off_gs, off_pieces, off_piece_strip;
};

inline size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

struct Q4ListLayout {
    size_t off_items, off_gs, off_pieces, off_piece_strip, total;
};
Q4ListLayout list_layout(int count, size_t total_groups, int nwarps) {
    Q4ListLayout L;
    L.off_items = align256(sizeof(Q4ListHeader));
    L.off_gs = align256(L.off_items + size_t(count) * sizeof(Q4Item));
    L.off_pieces = align256(L.off_gs + total_groups * 64);
    L.off_piece_strip = align256(L.off_pieces + size_t(nwarps) * 2 * kPieceFloats * 4);
    L.total = align256(L.off_piece_strip + size_t(nwarps) * 2 * 4);
    return L;
}

// Item that holds element `v` of a sequence whose per-item begins are read by `begin_of` (begins ascend).
template <typename F>
__device__ __forceinline__ int find_item(int count, uint32_t v, F begin_of) {
    int lo = 0, hi = count;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (begin_of(mid) <= v) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(256) k_q4_list_prepare(unsigned char* __restrict__ ws) {
    pdl_release();
    pdl_wait();  // the activations may come from the preceding kernel
    const Q4ListHeader* H = reinterpret_cast<const Q4ListHeader*>(ws);
    const Q4Item* items = reinterpret_cast<const Q4Item*>(ws + H->off_items);
    float2* gs = reinterpret_cast<float2*>(ws + H->off_gs);
    int32_t* piece_strip = reinterpret_cast<int32_t*>(ws + H->off_piece_strip);
    const int G = H->G, sub = threadIdx.x & 7;
    // the matrices' first groups go to shared memory: the search below would otherwise be a chain of
    // dependent loads from L2 that is most of this kernel's time
    __shared__ uint32_t group_begin_sm[TETRA_Q4_LIST_MAX];
    for (int i = threadIdx.x; i < H->count; i += blockDim.x) group_begin_sm[i] = items[i].group_begin;
    __syncthreads();
    for (uint32_t gg = (blockIdx.x * blockDim.x + threadIdx.x) >> 3; gg < H->total_groups;
         gg += (gridDim.x * blockDim.x) >> 3) {
        const int it = find_item(H->count, gg, [&](int i) { return group_begin_sm[i]; });
        const uint2* src = reinterpret_cast<const uint2*>(items[it].x + size_t(gg - items[it].group_begin) * G);
        float lo = 0.f, hi = 0.f;  // k % 4 in {0, 1} / {2, 3}
        for (int i = 0; i < G / 32; ++i) {
            const uint2 u = __ldg(src + sub + 8 * i);
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&u.x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
            lo += a.x + a.y;
            hi += b.x + b.y;
        }
#pragma unroll
        for (int o = 4; o >= 1; o >>= 1) {
            lo += __shfl_xor_sync(0xFFFFFFFFu, lo, o);
            hi += __shfl_xor_sync(0xFFFFFFFFu, hi, o);
        }
        // eight (sum x, -sum bias x) pairs per group, one per MMA column; only column 0 carries a vector
        gs[size_t(gg) * 8 + sub] = sub == 0 ? make_float2(lo + hi, -(1024.f * lo + 64.f * hi)) : make_float2(0.f, 0.f);
    }
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < 2 * H->nwarps; i += gridDim.x * blockDim.x) piece_strip[i] = -1;
}

template <int G, int DEPTH>
__global__ void __launch_bounds__(kQ4ListThreads, 1) k_q4_list_main(unsigned char* __restrict__ ws) {
    constexpr int TPG = G / 64, CH = q4_chunk_bytes(G), PIECES = CH / 16;
    extern __shared__ __align__(16) unsigned char q4_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    pdl_release();
    // the plan (written once, long before) and the weights do not depend on the preceding kernel
    const Q4ListHeader* H = reinterpret_cast<const Q4ListHeader*>(ws);
    const Q4Item* items = reinterpret_cast<const Q4Item*>(ws + H->off_items);
    const unsigned char* gs = ws + H->off_gs;
    float* pieces = reinterpret_cast<float*>(ws + H->off_pieces);
    int32_t* piece_strip = reinterpret_cast<int32_t*>(ws + H->off_piece_strip);
    const int gw = blockIdx.x * kQ4ListWarps + warp, nw = gridDim.x * kQ4ListWarps;
    const uint32_t c_begin = uint32_t(uint64_t(H->total_chunks) * gw / nw);
    const uint32_t c_end = uint32_t(uint64_t(H->total_chunks) * (gw + 1) / nw);
    if (c_begin >= c_end) return;

    const uint32_t ring_lane = smem_u32(q4_smem) + uint32_t(warp) * (DEPTH * CH) + lane * 16;
    const uint32_t ring_lane_end = ring_lane + DEPTH * CH;
    const bool tail_lane = lane < PIECES % 32;  // lanes that copy the last, partial group of 16-byte pieces

    // fetch side: the next chunk to copy, wherever in the list it lies
    int fi = find_item(H->count, c_begin, [&](int i) { return items[i].chunk_begin; });
    uint32_t f_left_in_item = items[fi].chunk_begin + uint32_t(items[fi].groups) * uint32_t(items[fi].strips) - c_begin;
    const unsigned char* f_src = items[fi].packed + size_t(c_begin - items[fi].chunk_begin) * CH + lane * 16;
    int f_todo = int(c_end - c_begin);
    auto fetch_into = [&](uint32_t dst_lane) {
        if (f_todo > 0) {
#pragma unroll
            for (int i = 0; i < PIECES / 32; ++i) q4_cp_async16(dst_lane + i * 512, f_src + i * 512);
            if (PIECES % 32 != 0 && tail_lane) q4_cp_async16(dst_lane + (PIECES / 32) * 512, f_src + (PIECES / 32) * 512);
            f_src += CH;
            if (--f_left_in_item == 0 && f_todo > 1) {  // on to the next matrix of the list
                ++fi;
                f_src = items[fi].packed + lane * 16;
                f_left_in_item = uint32_t(items[fi].groups) * uint32_t(items[fi].strips);
            }
        }
        --f_todo;
        asm volatile("cp.async.commit_group;" ::: "memory");  // one group per call, empty or not
    };
#pragma unroll
    for (int i = 0; i < DEPTH - 1; ++i) fetch_into(ring_lane + i * CH);

    pdl_wait();  // the group sums come from k_q4_list_prepare, the activations possibly from a kernel before it

    uint32_t slot_lane = ring_lane;                       // slot being consumed
    uint32_t refill_lane = ring_lane + (DEPTH - 1) * CH;  // slot consumed last (empty at the start)
    const uint32_t so_delta = uint32_t(TPG * 1024 + g * 4) - uint32_t(lane * 16);  // slot_lane -> this lane's scale records

    // consume side
    int ci = find_item(H->count, c_begin, [&](int i) { return items[i].chunk_begin; });
    uint32_t left = c_end - c_begin;
    uint32_t local = c_begin - items[ci].chunk_begin;  // chunk index inside matrix ci
    int n_pieces = 0;
    while (left > 0) {
        const Q4Item I = items[ci];
        const int groups = I.groups;
        int strip = int(local / uint32_t(groups));
        int gi = int(local - uint32_t(strip) * uint32_t(groups));
        uint32_t in_item = min(left, uint32_t(groups) * uint32_t(I.strips) - local);
        left -= in_item;
        local += in_item;
        // column 0 of the B fragment is the activation vector; the other columns repeat it and are never stored
        const __half* x_lane = I.x + 16 * t;
        const unsigned char* gs_lane = gs + size_t(I.group_begin) * 64 + t * 16;
        while (in_item > 0) {
            // one segment: the chunks of this warp that belong to one strip
            const int seg_first = gi;
            const uint32_t seg_len = min(uint32_t(groups - gi), in_item);
            float acc[2][4];
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[h][i] = 0.f;
            for (uint32_t c = 0; c < seg_len; ++c, ++gi) {
                const uint4 csv = __ldg(reinterpret_cast<const uint4*>(gs_lane + size_t(gi) * 64));
                const uint32_t cs[4] = {csv.x, csv.y, csv.z, csv.w};  // (sum x, -sum bias x) of columns 2 t, 2 t + 1
                fetch_into(refill_lane);
                q4_cp_async_wait<DEPTH - 1>();  // this chunk has landed
                __syncwarp();
                float d[2][4];
#pragma unroll
                for (int j = 0; j < TPG; ++j) {
                    const uint4* xg = reinterpret_cast<const uint4*>(x_lane + size_t(gi) * G) + 8 * j;  // L1-resident
                    const uint4 xa = __ldg(xg);
                    const uint4 xb = __ldg(xg + 1);
                    const uint32_t xr[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
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
                const float sx_even = __uint_as_float(cs[0]), sx_odd = __uint_as_float(cs[2]);
                const uint32_t so_lane = slot_lane + so_delta;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t so0 = lds32(so_lane + 64 * h);
                    const uint32_t so1 = lds32(so_lane + 64 * h + 32);
                    const float2 r0 = __half22float2(*reinterpret_cast<const __half2*>(&so0));  // (scale, offset)
                    const float2 r1 = __half22float2(*reinterpret_cast<const __half2*>(&so1));
                    fma2(r0.y, sx_even, sx_odd, acc[h][0], acc[h][1]);
                    fma2(r0.x, d[h][0], d[h][1], acc[h][0], acc[h][1]);
                    fma2(r1.y, sx_even, sx_odd, acc[h][2], acc[h][3]);
                    fma2(r1.x, d[h][2], d[h][3], acc[h][2], acc[h][3]);
                }
                __syncwarp();  // every lane has read the slot before the next refill targets it
                refill_lane = slot_lane;
                slot_lane += CH;
                if (slot_lane == ring_lane_end) slot_lane = ring_lane;
            }
            in_item -= seg_len;
            // element 8 lane + 4 h + i is (row 16 h + g + 8 (i / 2), column 2 t + (i % 2)) of the strip
            if (seg_first == 0 && gi == groups) {  // the whole strip was this warp's: store column 0
                if (t == 0) {
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int i = 0; i < 4; i += 2) {
                            const int row = 32 * strip + 16 * h + g + 8 * (i >> 1);
                            if (row < I.N) I.y[row] = acc[h][i];
                        }
                }
            } else {  // a strip shared with a neighbouring warp: leave a piece (column 0: row 16 h + g + 8 j at 4 g' ...)
                if (t == 0) {  // floats 4 g .. 4 g + 3 = rows g, g + 8, 16 + g, 24 + g
                    float* mine = pieces + size_t(2 * gw + n_pieces) * kPieceFloats + 4 * g;
                    *reinterpret_cast<float4*>(mine) = make_float4(acc[0][0], acc[0][2], acc[1][0], acc[1][2]);
                }
                if (lane == 0) piece_strip[2 * gw + n_pieces] = int32_t(I.strip_begin) + strip;
                ++n_pieces;
            }
            if (gi == groups) {
                gi = 0;
                ++strip;
            }
        }
        ++ci;
        local = 0;
    }
    q4_cp_async_wait<0>();
}

// Warp i looks at piece slot i (slots are in memory order: warp, then first/second): if it holds the first
// piece of its strip, the warp adds the strip's pieces in slot order and stores the 32 rows.
__global__ void __launch_bounds__(256) k_q4_list_combine(unsigned char* __restrict__ ws) {
    pdl_release();
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    pdl_wait();
    const Q4ListHeader* H = reinterpret_cast<const Q4ListHeader*>(ws);
    const int npieces = 2 * H->nwarps;
    if (i >= npieces) return;
    const int32_t* piece_strip = reinterpret_cast<const int32_t*>(ws + H->off_piece_strip);
    const int sid = piece_strip[i];
    if (sid < 0) return;
    // a strip has at most one piece per warp: its earlier pieces, if any, sit in the slots just before
    int j = i - 1;
    while (j >= 0 && piece_strip[j] < 0) --j;
    if (j >= 0 && piece_strip[j] == sid) return;  // not the first piece of its strip
    const float* pieces = reinterpret_cast<const float*>(ws + H->off_pieces);
    float total = 0.f;
    for (int k = i; k < npieces; ++k) {
        const int s = piece_strip[k];
        if (s < 0) continue;
        if (s != sid) break;
        total += pieces[size_t(k) * kPieceFloats + lane];
    }
    const Q4Item* items = reinterpret_cast<const Q4Item*>(ws + H->off_items);
    const int it = find_item(H->count, uint32_t(sid), [&](int q) { return items[q].strip_begin; });
    // float 4 g + j of a piece is row g + 8 (j & 1) + 16 (j >> 1) of the strip
    const int g = lane >> 2, jj = lane & 3;
    const int row = 32 * (sid - int(items[it].strip_begin)) + g + 8 * (jj & 1) + 16 * (jj >> 1);
    if (row < items[it].N) items[it].y[row] = total;
}

int check_list(const tetra_q4_problem* p, int count, int G) {
    if (!p) return TETRA_ERR_NULL;
    if (count <= 0 || count > TETRA_Q4_LIST_MAX) return TETRA_ERR_SHAPE;
    if (G != 64 && G != 128) return TETRA_ERR_SHAPE;
    for (int i = 0; i < count; ++i) {
        if (!p[i].packed || !p[i].x || !p[i].y) return TETRA_ERR_NULL;
        if (p[i].N <= 0 || p[i].K <= 0 || p[i].K > TETRA_Q4_MAX_K || p[i].K % G) return TETRA_ERR_SHAPE;
        if ((reinterpret_cast<uintptr_t>(p[i].packed) & 15) || (reinterpret_cast<uintptr_t>(p[i].x) & 15) ||
            (reinterpret_cast<uintptr_t>(p[i].y) & 3))
            return TETRA_ERR_ALIGN;
    }
    return TETRA_OK;
}

template <int G, int DEPTH>
cudaError_t run_main(unsigned char* ws, int sms, cudaStream_t s) {
    const size_t smem = size_t(kQ4ListWarps) * DEPTH * q4_chunk_bytes(G);
    static PerDeviceOnce once;
    cudaError_t e = once.run([smem] {
        return cudaFuncSetAttribute(k_q4_list_main<G, DEPTH>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    });
    if (e != cudaSuccess) return e;
    return launch_pdl(k_q4_list_main<G, DEPTH>, sms, kQ4ListThreads, smem, s, ws);
}

}  // namespace
}  // namespace tetra

using namespace tetra;

extern "C" {

size_t tetra_q4_list_workspace_bytes(const tetra_q4_problem* problems_host, int count, int G) {
    if (check_list(problems_host, count, G) != TETRA_OK) return 0;
    int sms = 0;
    if (device_sms(&sms) != cudaSuccess) return 0;
    size_t groups = 0;
    for (int i = 0; i < count; ++i) groups += size_t(problems_host[i].K / G);
    return list_layout(count, groups, sms * kQ4ListWarps).total;
}

int tetra_q4_list_plan(const tetra_q4_problem* problems_host, int count, int G, void* workspace_dev,
                       size_t workspace_bytes, void* stream) {
    const int rc = check_list(problems_host, count, G);
    if (rc != TETRA_OK) return rc;
    if (!workspace_dev) return TETRA_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 255) return TETRA_ERR_ALIGN;
    int sms = 0;
    if (device_sms(&sms) != cudaSuccess) return TETRA_ERR_CUDA;
    const int nwarps = sms * kQ4ListWarps;
    uint64_t chunks = 0, groups = 0, strips = 0;
    for (int i = 0; i < count; ++i) {
        const uint64_t gr = uint64_t(problems_host[i].K / G), st = uint64_t((problems_host[i].N + 31) / 32);
        chunks += gr * st;
        groups += gr;
        strips += st;
    }
    if (chunks > 0x7FFFFFF0ull || strips > 0x7FFFFFF0ull) return TETRA_ERR_SHAPE;
    const Q4ListLayout L = list_layout(count, size_t(groups), nwarps);
    if (workspace_bytes < L.total) return TETRA_ERR_SIZE;
    const size_t meta = L.off_gs;
    unsigned char* buf = static_cast<unsigned char*>(std::calloc(1, meta));
    if (!buf) return TETRA_ERR_CUDA;
    Q4ListHeader* H = reinterpret_cast<Q4ListHeader*>(buf);
    H->count = count;
    H->G = G;
    H->nwarps = nwarps;
    H->total_chunks = uint32_t(chunks);
    H->total_groups = uint32_t(groups);
    H->total_strips = uint32_t(strips);
    H->off_items = uint32_t(L.off_items);
    H->off_gs = uint32_t(L.off_gs);
    H->off_pieces = uint32_t(L.off_pieces);
    H->off_piece_strip = uint32_t(L.off_piece_strip);
    Q4Item* items = reinterpret_cast<Q4Item*>(buf + L.off_items);
    uint32_t cb = 0, gb = 0, sb = 0;
    for (int i = 0; i < count; ++i) {
        const tetra_q4_problem& q = problems_host[i];
        Q4Item& I = items[i];
        I.packed = static_cast<const unsigned char*>(q.packed);
        I.x = static_cast<const __half*>(q.x);
        I.y = q.y;
        I.N = q.N;
        I.K = q.K;
        I.groups = q.K / G;
        I.strips = (q.N + 31) / 32;
        I.chunk_begin = cb;
        I.group_begin = gb;
        I.strip_begin = sb;
        cb += uint32_t(I.groups) * uint32_t(I.strips);
        gb += uint32_t(I.groups);
        sb += uint32_t(I.strips);
    }
    // pageable source: the runtime has taken its copy when the call returns, so the buffer can be freed
    const cudaError_t e = cudaMemcpyAsync(workspace_dev, buf, meta, cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream));
    std::free(buf);
    return e == cudaSuccess ? TETRA_OK : TETRA_ERR_CUDA;
}

int tetra_q4_list_run(void* workspace_dev, int G, void* stream) {
    if (!workspace_dev) return TETRA_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 255) return TETRA_ERR_ALIGN;
    if (G != 64 && G != 128) return TETRA_ERR_SHAPE;
    int sms = 0;
    if (device_sms(&sms) != cudaSuccess) return TETRA_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned char* ws = static_cast<unsigned char*>(workspace_dev);
    cudaError_t e = launch_pdl(k_q4_list_prepare, sms * 2, 256, 0, s, ws);
    if (e == cudaSuccess) e = G == 128 ? run_main<128, 2>(ws, sms, s) : run_main<64, 6>(ws, sms, s);
    if (e == cudaSuccess) e = launch_pdl(k_q4_list_combine, (2 * sms * kQ4ListWarps + 7) / 8, 256, 0, s, ws);  // a warp per piece slot
    return e == cudaSuccess ? TETRA_OK : TETRA_ERR_CUDA;
}

}  // extern "C"
