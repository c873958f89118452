// tetra_gemv_noalloc: the decode-and-multiply product for callers that cannot
// allocate device memory.
//
// Some code that wants a Tetra product runs where cudaMalloc is off limits: a
// plug-in loaded into a host application that owns the memory pool and hands
// out no more, a real-time loop that must not take the allocator's lock, a
// process whose memory budget was fixed at start-up.  The planned-list kernels
// need a scratch area (the plan of the product plus the fixed-point image of the
// activations); here that area is a fixed array inside the library's own device
// image, so the call needs no buffer beyond its inputs and its output.
#include <mutex>

#include "../../include/tetra.h"
#include "tetra_launch.h"

using namespace tetra;

namespace {

constexpr int kNoAllocMaxBlocks = TETRA_NOALLOC_MAX_K / 24;         // words per row
constexpr size_t kNoAllocScratchBytes = 256 + size_t(kNoAllocMaxBlocks) * 80;

// Every GPU that loads the library holds this array until the process exits.
// Its name is a host-side handle, not a device address: the address a kernel
// can use comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Device address of the array on the current device (looked up on the first call there).
int scratch_address(void** out) {
    static void* address[64] = {nullptr};
    static std::mutex mu;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return TETRA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!address[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return TETRA_ERR_CUDA;
        address[dev] = p;
    }
    *out = address[dev];
    return TETRA_OK;
}

// The plan of one product, passed to the device BY VALUE: kernel parameters are copied when the
// launch is enqueued (and, under stream capture, when the node is created), so nothing points at
// host memory that may be gone by the time the work runs.
struct PlanBlob {
    unsigned char bytes[256];
};

__global__ void k_write_plan(unsigned char* __restrict__ scratch, const PlanBlob blob) {
    for (unsigned i = threadIdx.x; i < sizeof(PlanBlob) / 4; i += blockDim.x)
        reinterpret_cast<uint32_t*>(scratch)[i] = reinterpret_cast<const uint32_t*>(blob.bytes)[i];
}

}  // namespace

extern "C" int tetra_gemv_noalloc(const void* codes, const float* row_scales, const void* table, const void* x,
                                  float* y, int N, int K, const void* tail, void* stream) {
    if (!codes || !row_scales || !table || !x || !y) return TETRA_ERR_NULL;
    if (N <= 0 || K <= 0) return TETRA_ERR_SHAPE;
    if (K > TETRA_NOALLOC_MAX_K) return TETRA_ERR_SIZE;  // the fixed scratch array holds no more columns
    if (!aligned(codes, 16) || !aligned(table, 16) || !aligned(row_scales, 4) || !aligned(y, 4) || !aligned(x, 2) ||
        (tail && !aligned(tail, 2)))
        return TETRA_ERR_ALIGN;
    // words per row, by the same rule as tetra_gemv_tail: a row must hold at least one word
    const int B = (tail || K % 24 == 0) ? K / 24 : (K + 23) / 24;
    if (B <= 0) return TETRA_ERR_SHAPE;
    const Problem problem{codes, row_scales, x, (K % 24) ? tail : nullptr, y, N, K};
    if (single_plan_scratch_bytes(B) > kNoAllocScratchBytes) return TETRA_ERR_SIZE;

    void* scratch = nullptr;
    const int rc = scratch_address(&scratch);
    if (rc != TETRA_OK) return rc;

    // The plan of this one product goes to the head of the array (written by a one-block kernel from
    // its own parameters); the pre-pass kernel then rewrites the activation records behind it.
    // Nothing in the array has to start at zero: every byte the kernels read is written by this call
    // first, whatever an earlier call left there.
    PlanBlob blob;
    static_assert(sizeof blob.bytes >= 256, "plan blob");
    if (single_plan_meta_bytes() > sizeof blob.bytes) return TETRA_ERR_SIZE;
    single_plan_fill(problem, blob.bytes);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    k_write_plan<<<1, 64, 0, s>>>(static_cast<unsigned char*>(scratch), blob);
    if (cudaGetLastError() != cudaSuccess) return TETRA_ERR_CUDA;
    return grouped_run(scratch, table, s) == cudaSuccess ? TETRA_OK : TETRA_ERR_CUDA;
}
