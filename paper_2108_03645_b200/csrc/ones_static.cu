// ones_select_top_noalloc: the top-e selection for callers that cannot provide scratch memory.
//
// Some users of this library run where device memory cannot be obtained at call time: a scheduler
// plug-in inside a process whose framework has already claimed the whole device (cudaMalloc fails
// there, and a caching allocator they do not own cannot be asked), or a round loop with a latency
// budget in which the implicit device-wide synchronisation of an allocation is not acceptable.
// For them the partial-result scratch of the selection lives in a fixed array that is part of
// this library's device image: every GPU that loads the library holds these 128 KiB until the
// process exits, whether or not the entry point is ever called.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "ones.h"
#include "ones_internal.h"

namespace {

constexpr int kMaxDevices = 64;
constexpr size_t kScratchBytes = (size_t)ones::kTopBlocksMax * ONES_NOALLOC_MAX_TOP * 16;  // 128 KiB

// Partial top-e lists of the selection's first stage (one list of e records per block).
// Host code must not hand this name to a kernel: on the host it is only a stand-in for the
// symbol; the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_top_scratch[kScratchBytes];

std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of g_top_scratch on the current device (looked up on the first call there).
cudaError_t scratch_address(void** out) {
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        err = cudaGetSymbolAddress((void**)&ptr, g_top_scratch);
        if (err != cudaSuccess) return err;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int ones_select_top_noalloc(const double* d_fitness, int32_t n, int32_t e, int32_t* d_index,
                                       void* cuda_stream) {
    if (!d_fitness || !d_index) return ONES_ERR_NULL;
    if (n <= 0 || e <= 0 || e > n) return ONES_ERR_BAD_PARAM;
    if (e > ONES_NOALLOC_MAX_TOP) return ONES_ERR_WORKSPACE;  // beyond the built-in scratch: use ones_select_top
    if (ones::top_scratch_bytes(n, e) > kScratchBytes) return ONES_ERR_WORKSPACE;
    void* scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return ONES_ERR_CUDA;
    // Nothing in the scratch has to start at zero: the first stage writes all e records of every
    // block it launches (empty ones included) before the second stage reads exactly those.
    cudaError_t err = ones::launch_top(d_fitness, n, e, d_index, scratch,
                                       reinterpret_cast<cudaStream_t>(cuda_stream), nullptr);
    return err == cudaSuccess ? ONES_OK : ONES_ERR_CUDA;
}
