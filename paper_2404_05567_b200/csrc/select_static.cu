// dsmoe_select_static: expert selection for callers that cannot allocate device memory.
//
// dsmoe_select needs a small scratch area (per-chunk expert counts) that its caller normally
// allocates.  Some callers cannot do that: code running inside a framework that owns the device
// allocator and forbids cudaMalloc on its streams, plugins loaded into a serving process that were
// handed only input and output buffers, or a latency-critical loop in which any allocation (and the
// implicit synchronisation it may bring) is off the table.  For them the scratch lives in a
// file-scope device array that the library itself carries; every GPU that loads the library holds
// these kStaticScratchBytes until the process exits.
#include "common.cuh"

namespace dsmoe {
namespace {

constexpr size_t kStaticScratchInts = 128 * 1024;                 // 512 KiB
constexpr size_t kStaticScratchBytes = kStaticScratchInts * sizeof(int32_t);
constexpr int kMaxDevices = 64;

// Device memory.  In host code this name is only a handle for cudaGetSymbolAddress -- it is NOT a
// device address, and passing it to a kernel would make the kernel read or write the wrong memory.
static __device__ __align__(256) int32_t g_select_scratch[kStaticScratchInts];

// Device address of g_select_scratch on each device, looked up once per device.
int32_t* g_scratch_ptr[kMaxDevices] = {};

dsmoe_status scratch_for_current_device(int32_t** out) {
    int dev = -1;
    DSMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return DSMOE_ERR_UNSUPPORTED;
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        DSMOE_CUDA_TRY(cudaGetSymbolAddress(&p, g_select_scratch));   // resolves the symbol on the current device
        if (!p) return DSMOE_ERR_CUDA;
        g_scratch_ptr[dev] = static_cast<int32_t*>(p);
    }
    *out = g_scratch_ptr[dev];
    return DSMOE_OK;
}

}  // namespace
}  // namespace dsmoe

using namespace dsmoe;

extern "C" dsmoe_status dsmoe_select_static(const dsmoe_layer_desc* desc, const float* scores, uint64_t* mask,
                                            int32_t* k_t, int32_t* counts, int32_t* offsets, dsmoe_stream stream) {
    DSMOE_TRY(check_desc(desc));
    if (!counts || !offsets) return DSMOE_ERR_INVALID_ARG;
    if (desc->T > 0 && (!scores || !mask || !k_t)) return DSMOE_ERR_INVALID_ARG;
    // scratch needed: one int32 per (chunk of 32 tokens, expert)
    const size_t need = (size_t)ceil_div(desc->T, kChunk) * (size_t)desc->E;
    if (need > kStaticScratchInts) return DSMOE_ERR_WORKSPACE;   // beyond the built-in scratch: use dsmoe_select
    int32_t* scratch = nullptr;
    DSMOE_TRY(scratch_for_current_device(&scratch));
    cudaStream_t s = (cudaStream_t)stream;
    // Nothing in the scratch has to start at zero: the counting kernel overwrites every entry it later reads,
    // so whatever the previous call left behind is never observed.
    DSMOE_TRY(launch_select(*desc, scores, mask, k_t, s));
    return launch_finalize(*desc, mask, counts, offsets, scratch, nullptr, s);
}
