// ardiff_entropy_gate_noalloc: the entropy gate + compaction for callers that must not allocate.
//
// Some hosts of this library cannot let it call cudaMalloc: a serving process that has handed the
// whole device to its own pool allocator, code that runs while a stream is being captured (where an
// allocation is an error), or a real-time loop that may not take the allocator's lock or the
// implicit device synchronisation an allocation can bring. The regular ardiff_entropy_gate
// allocates its small per-block count array on its first call on each device; this variant keeps
// that array in the library image instead, as a fixed-size __device__ array that every GPU loading
// the library holds until the process exits.
//
// The kernels, the launch shape rules and the results are those of ardiff_entropy_gate; only the
// origin of the scratch pointer differs.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/ardiff.h"
#include "common.cuh"

namespace {

constexpr int kStaticGateBlocks = ARDIFF_GATE_NOALLOC_MAX_BLOCKS;

// Per-block kept-token counts of the call in flight. 4 KB per device. Written in full by the
// entropy kernel (one entry per launched block) before the compaction kernel reads it, so nothing
// in it has to start at zero and a call never depends on what the previous call left behind.
static __device__ __align__(256) int32_t g_static_block_counts[kStaticGateBlocks];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
int32_t* g_static_ptr[kMaxDevices] = {nullptr};
int g_static_sms[kMaxDevices] = {0};

// In host code `g_static_block_counts` is only a handle for the symbol, never a device address:
// the address on the current device comes from cudaGetSymbolAddress, once per device.
int static_scratch(int32_t** ptr, int* sms) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ARDIFF_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return ARDIFF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_block_counts) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return ARDIFF_ERR_CUDA;
        }
        int n_sm = 0;
        if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1)
            return ARDIFF_ERR_CUDA;
        g_static_sms[dev] = n_sm;
        g_static_ptr[dev] = static_cast<int32_t*>(p);
    }
    *ptr = g_static_ptr[dev];
    *sms = g_static_sms[dev];
    return ARDIFF_OK;
}

}  // namespace

extern "C" int ardiff_entropy_gate_noalloc(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                                           int32_t* idx, int32_t* count, void* stream) {
    // the fixed capacity is checked before anything touches the device
    if (n < 0 || n > (int64_t)ARDIFF_GATE_NOALLOC_MAX_TOKENS) return ARDIFF_ERR_SHAPE;
    int32_t* counts = nullptr;
    int sms = 0;
    const int rc = static_scratch(&counts, &sms);
    if (rc != ARDIFF_OK) return rc;
    return ardiff::gate_launch(feat, n, d, tau, mask, idx, count, nullptr, counts, nullptr, nullptr,
                               kStaticGateBlocks, sms, static_cast<cudaStream_t>(stream));
}
