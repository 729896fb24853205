// Tensor-core (tcgen05) Stream mask kernel. Placeholder until the kernel lands.
#include "common.cuh"

namespace stream {
bool mask_tc_supported(const Geom &, int) { return false; }
stream_status launch_mask_tc(const Geom &, const void *, const void *, int32_t *, float *, WorkspaceHeader *, cudaStream_t) {
    set_error("tensor-core mask kernel not built");
    return STREAM_ERR_UNSUPPORTED;
}
}  // namespace stream
