// stream_build_mask_static: the mask build for callers that cannot hand over a workspace.
//
// Some hosts of this library cannot obtain device memory at call time: an inference engine that
// gives all of HBM to its own pool at start-up (a later cudaMalloc simply fails), or a
// latency-critical loop where the implicit device-wide synchronisation of cudaMalloc / cudaFree
// is not acceptable. For them the kernel's scratch (the 256-byte header with the work counter of
// the persistent kernel and the call's counters) lives in a file-scope device array that every
// GPU loading the library holds until the process exits.
#include <mutex>

#include "common.cuh"

namespace stream {
namespace {

constexpr size_t kStaticScratchBytes = 4096;  // the stated maximum; today's kernels need 256
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device. In host code the array's name is only a
// handle for the runtime, never a pointer a kernel may use: the address comes from
// cudaGetSymbolAddress, asked once per device with that device current.
stream_status scratch_for_current_device(void **out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) { set_error("device ordinal %d outside 0..%d", dev, kMaxDevices - 1); return STREAM_ERR_UNSUPPORTED; }
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_addr[dev] == nullptr) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        if (ptr == nullptr || ((uintptr_t)ptr & 255) != 0) { set_error("static scratch has no usable device address"); return STREAM_ERR_CUDA; }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return STREAM_OK;
}

}  // namespace
}  // namespace stream

extern "C" stream_status stream_build_mask_static(const stream_problem *p, const void *q, const void *k,
                                                  int32_t *mask_out, float *score_out, void *cuda_stream) {
    using namespace stream;
    const size_t need = stream_workspace_bytes(p);
    // 0: the problem is invalid or unsupported. The workspace variant validates the problem before it
    // looks at its workspace, so asking it gives exactly the status (and text) it would give.
    if (need == 0) return stream_build_mask(p, q, k, mask_out, score_out, nullptr, 0, cuda_stream);
    if (need > kStaticScratchBytes) {
        set_error("this problem needs %zu bytes of scratch, the built-in array holds %zu: use stream_build_mask with a workspace",
                  need, kStaticScratchBytes);
        return STREAM_ERR_WORKSPACE;
    }
    void *scratch = nullptr;
    stream_status rc = scratch_for_current_device(&scratch);
    if (rc != STREAM_OK) return rc;
    // Same path as the workspace variant from here on; it zeroes the header on the stream first.
    // (Just the header's bytes are handed over, which keeps the optional per-row counters off.)
    return stream_build_mask(p, q, k, mask_out, score_out, scratch, need, cuda_stream);
}
