// stream_selftest_bounded_wait: runs the bounded mbarrier wait of the tensor-core kernels to its
// limit once, on a barrier of its own that nothing ever arrives at, so that the path "wait ran
// out -> error word -> abort flag -> the warp leaves together -> the host reads
// STREAM_ERR_DEVICE_CHECK" can be exercised without touching a product kernel. One warp, no
// copies and no MMAs in flight, nothing to drain: the kernel simply returns.
#include "tc_common.cuh"

namespace stream {
namespace {

constexpr unsigned kSelftestCode = 901;

__global__ void __launch_bounds__(32) selftest_wait_kernel(WorkspaceHeader *ws, long long limit) {
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // phase 0 of a fresh barrier completes with its first arrival, and there is none
    const bool ok = tc::mbar_wait_warp(tc::smem_u32(&bar), 0u, &abort_flag, &ws->error, &ws->error_info, kSelftestCode, limit);
    // every lane got the same answer; `rows` says which, `tiles_scored` whether the flag was raised
    if (threadIdx.x == 0) {
        ws->rows = ok ? 1ull : 0ull;
        ws->tiles_scored = (unsigned long long)abort_flag;
    }
}

}  // namespace
}  // namespace stream

extern "C" stream_status stream_selftest_bounded_wait(int64_t limit_cycles, void *workspace, size_t workspace_bytes,
                                                      void *cuda_stream) {
    using namespace stream;
    if (limit_cycles < 1 || limit_cycles > (1ll << 31)) {
        set_error("limit_cycles must lie in 1 .. 2^31 (got %lld)", (long long)limit_cycles);
        return STREAM_ERR_INVALID_ARG;
    }
    if (workspace == nullptr || workspace_bytes < sizeof(WorkspaceHeader) || ((uintptr_t)workspace & 255) != 0) {
        set_error("workspace must be a 256-byte aligned device buffer of at least %zu bytes", sizeof(WorkspaceHeader));
        return STREAM_ERR_WORKSPACE;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemsetAsync(workspace, 0, sizeof(WorkspaceHeader), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(workspace)");
    selftest_wait_kernel<<<1, 32, 0, st>>>((WorkspaceHeader *)workspace, (long long)limit_cycles);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "selftest launch");
    return STREAM_OK;
}
