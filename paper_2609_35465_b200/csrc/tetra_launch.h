// Host-side launch functions shared between the translation units.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include <mutex>

namespace tetra {

// One-time set-up per device (function attributes and the like), safe when several host threads
// make their first call at once.
class PerDeviceOnce {
public:
    template <typename F>
    cudaError_t run(F&& setup) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mu_);
        if (!done_[dev]) {
            e = setup();
            if (e != cudaSuccess) return e;
            done_[dev] = true;
        }
        return cudaSuccess;
    }

private:
    static constexpr int kMaxDevices = 64;
    std::mutex mu_;
    bool done_[kMaxDevices] = {};
};


// Multiprocessors of the current device (cached per device, thread-safe).
cudaError_t device_sms(int* sms);

// Device-side view of one product; same layout as tetra_problem in tetra.h.
struct Problem {
    const void* codes;
    const float* row_scales;
    const void* x;
    const void* tail;
    float* y;
    int32_t N;
    int32_t K;
};
static_assert(sizeof(Problem) == 48, "Problem must match tetra_problem");

cudaError_t launch_decode_file(const void* codes, const void* table, int8_t* y, uint8_t* mg, size_t nblocks,
                               cudaStream_t s);
cudaError_t launch_pack(const void* codes, const void* table, void* packed, int N, int B, cudaStream_t s);
cudaError_t launch_decode_packed(const void* packed, const void* table, int8_t* y, uint8_t* mg, int N, int B,
                                 cudaStream_t s);

// Paper-design GEMV (warp per row, lane per block) on file-order words.
cudaError_t launch_gemv_paper(const void* codes, size_t row_stride, const float* row_scales, const void* table,
                              const void* x, float* y, int N, int K, int batch, const void* tail, cudaStream_t s);

// One matrix or a short list of matrices in a single launch, no scratch memory (the kernel behind
// tetra_gemv, tetra_gemv_tail and tetra_gemv_list).  `batch` activation vectors per matrix, x and y
// advanced by K and N per vector.
constexpr int kListMax = 8;
struct ListDesc {
    int32_t count;
    int32_t total_groups;               // eight-row groups of all matrices
    int32_t group_prefix[kListMax + 1]; // row groups before matrix i
    int32_t max_blocks;                 // largest number of words per row in the list
    Problem problems[kListMax];
};
cudaError_t launch_gemv_list(const ListDesc& list, int batch, const void* table, cudaStream_t s);

// Planned list of batch-1 products.  grouped_plan writes descriptors and prefix
// arrays to the workspace (once per list); grouped_run enqueues the activation
// pre-pass and the persistent GEMV kernel (every step).
size_t grouped_workspace_bytes(const Problem* problems_host, int count);
cudaError_t grouped_plan(const Problem* problems_host, int count, void* ws_dev, size_t ws_bytes, cudaStream_t s);
cudaError_t grouped_run(void* ws_dev, const void* table, cudaStream_t s);


// 1..16 activation vectors at once (decode once, tensor-core contraction per block); ws holds the partial
// results of the CTAs' column ranges: batched_workspace_bytes(N, words per row).
size_t batched_workspace_bytes(int N, int blocks_per_row);
cudaError_t launch_gemv_batched(const void* codes, const float* row_scales, const void* table, const void* x,
                                float* y, int N, int K, int batch, const void* tail, void* ws, cudaStream_t s);

// Encoder search: per block of 24 weights the codebook point of largest cosine and the gain bit.
cudaError_t launch_encode(const float* w, const float* sigma, const void* table, unsigned char* codes, float* cosine,
                          size_t nblocks, cudaStream_t s);

// Plan of a single product, for callers that bring their own scratch memory:
// single_plan_fill writes single_plan_meta_bytes() bytes of plan data to a host
// buffer; copied to the start of a scratch area of single_plan_scratch_bytes(blocks)
// bytes, it makes that area a valid argument of grouped_run.
size_t single_plan_meta_bytes();
size_t single_plan_scratch_bytes(int blocks_per_row);
void single_plan_fill(const Problem& problem, unsigned char* meta_host);

}  // namespace tetra
