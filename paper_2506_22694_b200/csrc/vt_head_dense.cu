// Batched-serving head (B > 16): dense contraction on tcgen05 tensor cores.  Placeholder until
// the tensor-core kernel lands: reports the shape as unsupported so callers fail loudly.
#include "vt_common.cuh"

namespace vt {

bool head_dense_supported(int32_t, int32_t, int32_t) { return false; }
size_t head_dense_scratch_bytes(int32_t, int32_t, int32_t) { return 0; }
cudaError_t launch_head_dense(const HeadArgs&, Ctrl*, uint8_t*, cudaStream_t) {
    return cudaErrorNotSupported;
}

}  // namespace vt
