// extern "C" boundary of the Tetra library: argument checks and launches only.
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "../../include/tetra.h"
#include "tetra_launch.h"
#include "tetra_tables.h"

using namespace tetra;

namespace {

constexpr int kMaxBlocksPerRow = 2048;  // K <= 49,152
constexpr int kBatchedMinVectors = 2;   // tetra_gemv_batched runs the tensor-core kernel from this many vectors on

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }
inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? TETRA_OK : TETRA_ERR_CUDA; }

// The tables depend only on the gains; the integer part is built once.
const DeviceTables* host_tables(int* rc) {
    static DeviceTables* cached = nullptr;
    static int cached_rc = 0;
    static std::once_flag once;
    std::call_once(once, [] {
        cached = static_cast<DeviceTables*>(std::malloc(sizeof(DeviceTables)));
        cached_rc = cached ? build_device_tables(cached, nullptr) : -100;
    });
    *rc = cached_rc;
    return cached;
}

int check_gemv(const void* codes, const float* row_scales, const void* table, const void* x, const float* y, int N,
               int K, int batch) {
    if (!codes || !row_scales || !table || !x || !y) return TETRA_ERR_NULL;
    if (N <= 0 || K <= 0) return TETRA_ERR_SHAPE;
    if (batch < 1 || batch > TETRA_MAX_BATCH) return TETRA_ERR_BATCH;
    if (!aligned(codes, 16) || !aligned(table, 16) || !aligned(row_scales, 4) || !aligned(y, 4) || !aligned(x, 2))
        return TETRA_ERR_ALIGN;
    return TETRA_OK;
}

}  // namespace

extern "C" {

const char* tetra_status_string(int status) {
    switch (status) {
        case TETRA_OK: return "ok";
        case TETRA_ERR_NULL: return "null pointer";
        case TETRA_ERR_SHAPE: return "shape out of range";
        case TETRA_ERR_ALIGN: return "misaligned pointer";
        case TETRA_ERR_BATCH: return "batch out of range";
        case TETRA_ERR_CUDA: return "CUDA error";
        case TETRA_ERR_SIZE: return "buffer too small";
        case TETRA_ERR_TABLE: return "table build failed";
        default: return "unknown status";
    }
}

size_t tetra_table_bytes(void) { return sizeof(DeviceTables); }

int tetra_table_export(void* blob_host, size_t bytes) {
    if (!blob_host) return TETRA_ERR_NULL;
    if (bytes < size_t(TETRA_PAPER_TABLE_BYTES)) return TETRA_ERR_SIZE;
    int rc = 0;
    const DeviceTables* t = host_tables(&rc);
    if (rc) return TETRA_ERR_TABLE;
    std::memcpy(blob_host, &t->paper, sizeof(PaperTables));
    return TETRA_OK;
}

int tetra_build_table(void* table_dev, size_t bytes, const float* gain2_host, void* stream) {
    if (!table_dev) return TETRA_ERR_NULL;
    if (bytes < sizeof(DeviceTables)) return TETRA_ERR_SIZE;
    if (!aligned(table_dev, 16)) return TETRA_ERR_ALIGN;
    int rc = 0;
    const DeviceTables* base = host_tables(&rc);
    if (rc) return TETRA_ERR_TABLE;
    DeviceTables* t = static_cast<DeviceTables*>(std::malloc(sizeof(DeviceTables)));
    if (!t) return TETRA_ERR_TABLE;
    std::memcpy(t, base, sizeof(DeviceTables));
    if (gain2_host) {
        t->gain[0] = gain2_host[0];
        t->gain[1] = gain2_host[1];
        for (int g = 0; g < 2; ++g)
            for (int m = 0; m < 32; ++m) t->scale[0][m][2 * g] = -(t->gain[g] * t->paper.rsqrt16m[m]);
    }
    cudaError_t e = cudaMemcpyAsync(table_dev, t, sizeof(DeviceTables), cudaMemcpyHostToDevice, as_stream(stream));
    if (e == cudaSuccess) e = cudaStreamSynchronize(as_stream(stream));
    std::free(t);
    return cuda_status(e);
}

int tetra_decode_blocks(const void* codes_dev, const void* table_dev, int8_t* y_dev, uint8_t* mg_dev, size_t nblocks,
                        void* stream) {
    if (nblocks == 0) return TETRA_OK;  // nothing to do; empty buffers may be NULL
    if (!codes_dev || !table_dev || !y_dev) return TETRA_ERR_NULL;
    if (!aligned(codes_dev, 2) || !aligned(y_dev, 4) || !aligned(table_dev, 16)) return TETRA_ERR_ALIGN;
    return cuda_status(launch_decode_file(codes_dev, table_dev, y_dev, mg_dev, nblocks, as_stream(stream)));
}

size_t tetra_codes_bytes(int N, int nblocks) {
    if (N <= 0 || nblocks <= 0) return 0;
    return size_t((N + 7) / 8) * 48u * size_t(nblocks);
}

int tetra_pack_codes(const void* codes_dev, const void* table_dev, void* packed_dev, int N, int nblocks,
                     void* stream) {
    if (!codes_dev || !table_dev || !packed_dev) return TETRA_ERR_NULL;
    if (N <= 0 || nblocks <= 0 || nblocks > kMaxBlocksPerRow) return TETRA_ERR_SHAPE;
    if (!aligned(codes_dev, 2) || !aligned(packed_dev, 16) || !aligned(table_dev, 16)) return TETRA_ERR_ALIGN;
    return cuda_status(launch_pack(codes_dev, table_dev, packed_dev, N, nblocks, as_stream(stream)));
}

int tetra_decode_packed(const void* packed_dev, const void* table_dev, int8_t* y_dev, uint8_t* mg_dev, int N,
                        int nblocks, void* stream) {
    if (!packed_dev || !table_dev || !y_dev) return TETRA_ERR_NULL;
    if (N <= 0 || nblocks <= 0 || nblocks > kMaxBlocksPerRow) return TETRA_ERR_SHAPE;
    if (!aligned(packed_dev, 16) || !aligned(y_dev, 4) || !aligned(table_dev, 16)) return TETRA_ERR_ALIGN;
    return cuda_status(launch_decode_packed(packed_dev, table_dev, y_dev, mg_dev, N, nblocks, as_stream(stream)));
}

int tetra_gemv_tail(const void* codes, const float* row_scales, const void* table, const void* x, float* y, int N,
                    int K, int batch, const void* tail, void* stream) {
    const int rc = check_gemv(codes, row_scales, table, x, y, N, K, batch);
    if (rc) return rc;
    if (tail && !aligned(tail, 2)) return TETRA_ERR_ALIGN;
    const bool tail_mode = tail != nullptr || K % 24 == 0;
    const int B = tail_mode ? K / 24 : (K + 23) / 24;
    if (B <= 0 || B > kMaxBlocksPerRow) return TETRA_ERR_SHAPE;
    ListDesc list{};
    list.count = 1;
    list.total_groups = (N + 7) / 8;
    list.group_prefix[0] = 0;
    list.group_prefix[1] = list.total_groups;
    list.max_blocks = B;
    list.problems[0] = Problem{codes, row_scales, x, (K % 24) ? tail : nullptr, y, N, K};
    return cuda_status(launch_gemv_list(list, batch, table, as_stream(stream)));
}

int tetra_gemv(const void* codes, const float* row_scales, const void* table, const void* x, float* y, int N, int K,
               int batch, void* stream) {
    return tetra_gemv_tail(codes, row_scales, table, x, y, N, K, batch, nullptr, stream);
}

static int check_problems(const tetra_problem* problems_host, int count) {
    static_assert(sizeof(tetra_problem) == sizeof(Problem), "descriptor layouts must agree");
    if (!problems_host) return TETRA_ERR_NULL;
    if (count <= 0 || count > 65536) return TETRA_ERR_SHAPE;
    for (int i = 0; i < count; ++i) {
        const tetra_problem& q = problems_host[i];
        if (!q.codes || !q.row_scales || !q.x || !q.y) return TETRA_ERR_NULL;
        if (q.N <= 0 || q.K <= 0) return TETRA_ERR_SHAPE;
        if (!aligned(q.codes, 16) || !aligned(q.row_scales, 4) || !aligned(q.y, 4) || !aligned(q.x, 2) ||
            (q.tail && !aligned(q.tail, 2)))
            return TETRA_ERR_ALIGN;
        const int B = (q.tail || q.K % 24 == 0) ? q.K / 24 : (q.K + 23) / 24;
        if (B <= 0 || B > kMaxBlocksPerRow) return TETRA_ERR_SHAPE;
    }
    return TETRA_OK;
}

int tetra_gemv_list(const tetra_problem* problems_host, int count, const void* table, void* stream) {
    if (!table) return TETRA_ERR_NULL;
    if (!aligned(table, 16)) return TETRA_ERR_ALIGN;
    const int rc = check_problems(problems_host, count);
    if (rc) return rc;
    if (count > TETRA_LIST_MAX) return TETRA_ERR_SHAPE;
    ListDesc list{};
    list.count = count;
    long long groups = 0;
    for (int i = 0; i < count; ++i) {
        const tetra_problem& q = problems_host[i];
        list.group_prefix[i] = int32_t(groups);
        groups += (q.N + 7) / 8;
        const int B = (q.tail || q.K % 24 == 0) ? q.K / 24 : (q.K + 23) / 24;
        if (B > list.max_blocks) list.max_blocks = B;
        list.problems[i] = Problem{q.codes, q.row_scales, q.x, (q.K % 24) ? q.tail : nullptr, q.y, q.N, q.K};
    }
    if (groups > 0x7FFFFFF0LL) return TETRA_ERR_SHAPE;
    for (int i = count; i <= kListMax; ++i) list.group_prefix[i] = int32_t(groups);
    list.total_groups = int32_t(groups);
    return cuda_status(launch_gemv_list(list, 1, table, as_stream(stream)));
}

size_t tetra_grouped_workspace_bytes(const tetra_problem* problems_host, int count) {
    if (check_problems(problems_host, count) != TETRA_OK) return 0;
    return grouped_workspace_bytes(reinterpret_cast<const Problem*>(problems_host), count);
}

int tetra_gemv_grouped_plan(const tetra_problem* problems_host, int count, void* workspace_dev,
                            size_t workspace_bytes, void* stream) {
    const int rc = check_problems(problems_host, count);
    if (rc) return rc;
    if (!workspace_dev) return TETRA_ERR_NULL;
    if (!aligned(workspace_dev, 16)) return TETRA_ERR_ALIGN;
    if (workspace_bytes < grouped_workspace_bytes(reinterpret_cast<const Problem*>(problems_host), count))
        return TETRA_ERR_SIZE;
    return cuda_status(grouped_plan(reinterpret_cast<const Problem*>(problems_host), count, workspace_dev,
                                    workspace_bytes, as_stream(stream)));
}

int tetra_gemv_grouped_run(void* workspace_dev, const void* table, void* stream) {
    if (!workspace_dev || !table) return TETRA_ERR_NULL;
    if (!aligned(workspace_dev, 16) || !aligned(table, 16)) return TETRA_ERR_ALIGN;
    return cuda_status(grouped_run(workspace_dev, table, as_stream(stream)));
}

int tetra_gemv_grouped(const tetra_problem* problems_host, int count, const void* table, void* workspace_dev,
                       size_t workspace_bytes, void* stream) {
    if (!table) return TETRA_ERR_NULL;
    if (!aligned(table, 16)) return TETRA_ERR_ALIGN;
    const int rc = tetra_gemv_grouped_plan(problems_host, count, workspace_dev, workspace_bytes, stream);
    if (rc) return rc;
    return tetra_gemv_grouped_run(workspace_dev, table, stream);
}

size_t tetra_batched_workspace_bytes(int N, int K) {
    return (N > 0 && K > 0) ? batched_workspace_bytes(N, (K + 23) / 24) : 0;
}

int tetra_gemv_batched(const void* codes, const float* row_scales, const void* table, const void* x, float* y, int N,
                       int K, int batch, const void* tail, void* workspace_dev, size_t workspace_bytes, void* stream) {
    const int rc = check_gemv(codes, row_scales, table, x, y, N, K, batch);
    if (rc) return rc;
    if (!workspace_dev) return TETRA_ERR_NULL;
    if (!aligned(workspace_dev, 16) || (tail && !aligned(tail, 2))) return TETRA_ERR_ALIGN;
    const bool tail_mode = tail != nullptr || K % 24 == 0;
    const int B = tail_mode ? K / 24 : (K + 23) / 24;
    if (B <= 0 || B > kMaxBlocksPerRow) return TETRA_ERR_SHAPE;
    if (workspace_bytes < batched_workspace_bytes(N, B)) return TETRA_ERR_SIZE;
    // One vector: the single-launch kernel is faster than the tensor-core paths' fixed costs (measured on
    // B200, 4096 x 12288: 11.6 us against 15.8 us for two vectors on the tensor cores).
    if (batch <= kBatchedMinVectors - 1)
        return tetra_gemv_tail(codes, row_scales, table, x, y, N, K, batch, tail, stream);
    return cuda_status(launch_gemv_batched(codes, row_scales, table, x, y, N, K, batch, (K % 24) ? tail : nullptr,
                                           workspace_dev, as_stream(stream)));
}

int tetra_encode_blocks(const float* w_dev, const float* sigma_dev, const void* table_dev, void* codes_dev,
                        float* cosine_dev, size_t nblocks, void* stream) {
    if (nblocks == 0) return TETRA_OK;
    if (!w_dev || !table_dev || !codes_dev) return TETRA_ERR_NULL;
    if (!aligned(w_dev, 4) || !aligned(table_dev, 16) || (sigma_dev && !aligned(sigma_dev, 4)) ||
        (cosine_dev && !aligned(cosine_dev, 4)))
        return TETRA_ERR_ALIGN;
    return cuda_status(launch_encode(w_dev, sigma_dev, table_dev, static_cast<unsigned char*>(codes_dev), cosine_dev,
                                     nblocks, as_stream(stream)));
}

int tetra_gemv_paper_design(const void* codes, size_t row_stride, const float* row_scales, const void* table,
                            const void* x, float* y, int N, int K, int batch, const void* tail, void* stream) {
    if (!codes || !row_scales || !table || !x || !y) return TETRA_ERR_NULL;
    if (N <= 0 || K <= 0) return TETRA_ERR_SHAPE;
    if (batch < 1 || batch > TETRA_MAX_BATCH) return TETRA_ERR_BATCH;
    if (!aligned(codes, 2) || (row_stride & 1) || !aligned(table, 16) || !aligned(x, 2) || !aligned(y, 4))
        return TETRA_ERR_ALIGN;
    const bool tail_mode = tail != nullptr || K % 24 == 0;
    const size_t B = tail_mode ? K / 24 : (K + 23) / 24;
    if (B == 0 || row_stride < 6 * B) return TETRA_ERR_SHAPE;
    return cuda_status(launch_gemv_paper(codes, row_stride, row_scales, table, x, y, N, K, batch,
                                         (K % 24) ? tail : nullptr, as_stream(stream)));
}

int tetra_gemv_hostio(const void* codes, const float* row_scales, const void* table, const void* x_host,
                      float* y_host, void* x_stage_dev, float* y_stage_dev, int N, int K, int batch, const void* tail,
                      void* stream) {
    if (!x_host || !y_host || !x_stage_dev || !y_stage_dev) return TETRA_ERR_NULL;
    const int rc = check_gemv(codes, row_scales, table, x_stage_dev, y_stage_dev, N, K, batch);
    if (rc) return rc;
    cudaStream_t s = as_stream(stream);
    cudaError_t e = cudaMemcpyAsync(x_stage_dev, x_host, size_t(batch) * K * 2, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return TETRA_ERR_CUDA;
    const int rc2 = tetra_gemv_tail(codes, row_scales, table, x_stage_dev, y_stage_dev, N, K, batch, tail, stream);
    if (rc2) return rc2;
    e = cudaMemcpyAsync(y_host, y_stage_dev, size_t(batch) * N * sizeof(float), cudaMemcpyDeviceToHost, s);
    return cuda_status(e);
}

int tetra_gemv_grouped_hostio(void* workspace_dev, const void* table, const void* x_host, void* x_dev,
                              size_t x_bytes, float* y_host, const float* y_dev, size_t y_bytes, void* stream) {
    if (!workspace_dev || !table || !x_host || !x_dev) return TETRA_ERR_NULL;
    const bool mapped_results = !y_host && !y_dev;  // the plan's y pointers aim at page-locked host memory
    if (!mapped_results && (!y_host || !y_dev)) return TETRA_ERR_NULL;
    if (x_bytes == 0 || (!mapped_results && y_bytes == 0)) return TETRA_ERR_SIZE;
    if (!aligned(workspace_dev, 16) || !aligned(table, 16)) return TETRA_ERR_ALIGN;
    cudaStream_t s = as_stream(stream);
    if (cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return TETRA_ERR_CUDA;
    const int rc = tetra_gemv_grouped_run(workspace_dev, table, stream);
    if (rc || mapped_results) return rc;
    return cuda_status(cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, s));
}

}  // extern "C"
