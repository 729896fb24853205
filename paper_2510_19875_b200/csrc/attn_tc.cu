// Tensor-core block-sparse attention kernel. Placeholder until the kernel lands.
#include "common.cuh"

namespace stream {
bool attn_tc_supported(const Geom &, int) { return false; }
stream_status launch_attn_tc(const Geom &, const void *, const void *, const void *, const int32_t *, float, void *, cudaStream_t) {
    set_error("tensor-core attention kernel not built");
    return STREAM_ERR_UNSUPPORTED;
}
}  // namespace stream
