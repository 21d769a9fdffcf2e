// vt_select_topk_static: the top-K vocabulary selection for callers that cannot provide scratch.
//
// Some hosts of this library cannot hand over a workspace: a plugin that runs inside another
// framework's memory pool and must not go behind it, a process whose device memory was carved up
// completely at start-up, a callback that runs where the CUDA allocator may not be entered (a
// host function enqueued in a stream, for one).  For them the scratch of the selection
// kernel lives in a fixed device array that is part of the loaded library image: it costs
// VT_STATIC_SELECT_MAX_V * 16 bytes on every GPU that loads the library, for the life of the
// process, and it bounds the vocabulary this entry point accepts.
#include <mutex>

#include "vt_common.cuh"

namespace vt {
namespace {

constexpr size_t kSegWords = VT_STATIC_SELECT_MAX_V;            // one uint32 per id and array
// four arrays (keys and ids, ping and pong) of the radix sort behind the selection
static __device__ __align__(256) uint32_t g_select_scratch[4 * kSegWords];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
uint8_t* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device.  The name `g_select_scratch` means nothing
// to the GPU when used from host code -- it is the host-side handle of the symbol -- so the real
// address is looked up once per device, with that device current, and cached.
cudaError_t scratch_address(uint8_t** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_select_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = static_cast<uint8_t*>(p);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

thread_local cudaError_t t_last = cudaSuccess;

}  // namespace
}  // namespace vt

extern "C" vt_status vt_select_topk_static(const uint32_t* counts, int32_t V, int32_t K, int32_t* map,
                                           int32_t* inv_map, void* stream) {
    using namespace vt;
    if (!counts || !map || !inv_map || V < 1 || K < 1 || K > V) return VT_ERR_INVALID_ARG;
    if (V > VT_STATIC_SELECT_MAX_V) return VT_ERR_UNSUPPORTED;      // larger than the built-in scratch
    uint8_t* scratch = nullptr;
    cudaError_t e = scratch_address(&scratch);
    if (e != cudaSuccess) { t_last = e; return VT_ERR_CUDA; }
    // The launcher lays its four arrays out at multiples of align_up(V * 4, 256) <= kSegWords * 4
    // bytes; every word it reads was written earlier in the same launch, so nothing needs clearing.
    e = launch_select_topk(counts, V, K, map, inv_map, scratch, reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { t_last = e; return VT_ERR_CUDA; }
    return VT_OK;
}
