// stream_selftest_bounded_wait: runs the bounded mbarrier wait of the tensor-core kernels to its
// limit once, on a barrier of its own that nothing ever arrives at, so that the path "wait ran
// out -> error word -> abort flag -> the warp leaves together -> the host reads
// STREAM_ERR_DEVICE_CHECK" can be exercised without touching a product kernel. One warp, no
// copies and no MMAs in flight, nothing to drain: the kernel simply returns.
//
// stream_probe_unit_rates: two measurements of the SM units the tensor-core kernels lean on,
// taken on the device at hand so that a throughput figure can be set against what the hardware
// delivers: how fast two issuing warps bring L2-resident data into one SM's shared memory through
// TMA (one warp's copy stream alone stops at about 47 bytes per clock, two reach 77), and how long
// one tcgen05.mma of the mask kernel's shape (M = 128, N = 64, K = 16, bf16) occupies the tensor
// core when issued back to back.
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

// ---- unit rates ----------------------------------------------------------------------------------
constexpr int kProbeCopy = 16384;        // bytes per bulk copy
constexpr int kProbeBufs = 4;            // copies in flight per issuing warp
constexpr int kProbeWarps = 2;           // issuing warps (the mask kernel has two producer warps as well)
constexpr int kProbeSlice = 16;          // copies per CTA before its source slice repeats (256 KiB)
constexpr int kProbeCopies = 4096;       // copies per CTA
constexpr int kProbeChains = 2048;       // chains of eight MMAs
constexpr long long kProbeLimit = 1ll << 28;
constexpr unsigned kProbeCopyCode = 911, kProbeMmaCode = 912;
constexpr int kProbeSmem = kProbeWarps * kProbeBufs * kProbeCopy + 1024;   // copy buffers; the MMA operands reuse them

struct ProbeResult {  // in the first bytes of the scratch buffer
    unsigned long long copy_cycles, copy_bytes, mma_cycles, mma_count;
    unsigned int error, error_info;
};

// mode 0: both warps of every CTA keep kProbeBufs bulk copies of 16 KiB each in flight from the
// CTA's slice of `src` (L2-resident after the first pass); the rate is what the two bring together. mode 1: one lane of warp 0 issues chains of eight
// M = 128, N = 64, K = 16 MMAs on zero-filled operands into one TMEM slot. CTA 0 reports.
__global__ void __launch_bounds__(64) probe_rates_kernel(const unsigned char *src, ProbeResult *res, int mode) {
    extern __shared__ unsigned char probe_raw[];
    unsigned char *base = (unsigned char *)(((uintptr_t)probe_raw + 1023) & ~(uintptr_t)1023);
    __shared__ unsigned long long bars[kProbeWarps * kProbeBufs + 1];
    __shared__ unsigned long long warp_cycles[kProbeWarps];
    __shared__ unsigned int tmem_slot;
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < kProbeWarps * kProbeBufs * kProbeCopy / 16; i += blockDim.x) ((uint4 *)base)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        for (int i = 0; i <= kProbeWarps * kProbeBufs; ++i) tc::mbar_init(tc::smem_u32(&bars[i]), 1);
        for (int i = 0; i < kProbeWarps; ++i) warp_cycles[i] = 0ull;
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    tc::fence_async_smem();
    __syncthreads();
    if (mode == 1 && warp == 1) tc::tmem_alloc_512(tc::smem_u32(&tmem_slot));
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (warp < kProbeWarps && mode == 0) {
        const unsigned char *mine = src + (size_t)blockIdx.x * kProbeSlice * kProbeCopy;
        unsigned char *my_bufs = base + warp * kProbeBufs * kProbeCopy;
        long long t0, t1;
        asm volatile("mov.u64 %0, %%clock64;" : "=l"(t0)::"memory");
        bool ok = true;
        for (int i = 0; i < kProbeCopies + kProbeBufs && ok; ++i) {
            const int b = i % kProbeBufs;
            const unsigned bar = tc::smem_u32(&bars[warp * kProbeBufs + b]);
            // the copy that used this buffer last has landed
            if (i >= kProbeBufs) ok = tc::mbar_wait_warp(bar, ((i / kProbeBufs) - 1) & 1, &abort_flag, &res->error, &res->error_info, kProbeCopyCode, kProbeLimit);
            if (ok && i < kProbeCopies && tc::elect_one()) {
                tc::mbar_arrive_expect_tx(bar, kProbeCopy);
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(tc::smem_u32(my_bufs + b * kProbeCopy)), "l"(mine + (size_t)((i + warp * (kProbeSlice / 2)) % kProbeSlice) * kProbeCopy), "r"(kProbeCopy), "r"(bar) : "memory");
            }
            __syncwarp();
        }
        asm volatile("mov.u64 %0, %%clock64;" : "=l"(t1)::"memory");
        if (!ok) {  // give copies still in flight time to land before shared memory is handed back
            const long long w0 = clock64();
            while (clock64() - w0 < (1ll << 22)) { }
        }
        if (lane == 0 && ok) warp_cycles[warp] = (unsigned long long)(t1 - t0);
    } else if (warp == 0 && mode == 1) {
        const unsigned a_smem = tc::smem_u32(base), b_smem = a_smem + 2 * 128 * 128;  // A: [2 halves][128 rows][128 B]; B: [2][64][128 B]
        constexpr unsigned kHi = tc::desc_hi_sw128(1024);
        constexpr unsigned kI = tc::idesc_bf16(128, 64, false);
        const unsigned a_lo = tc::desc_lo_sw128(a_smem, 16), b_lo = tc::desc_lo_sw128(b_smem, 16);
        const unsigned done = tc::smem_u32(&bars[kProbeWarps * kProbeBufs]);
        const unsigned d_tmem = tmem_slot;
        long long t0, t1;
        asm volatile("mov.u64 %0, %%clock64;" : "=l"(t0)::"memory");
        if (tc::elect_one()) {
            for (int ch = 0; ch < kProbeChains; ++ch) {
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        tc::tc_mma_bf16_split(d_tmem, a_lo + ((c * 128 * 128 + k4 * 32) >> 4), kHi, b_lo + ((c * 64 * 128 + k4 * 32) >> 4), kHi, kI,
                                              (c | k4) != 0);
            }
            tc::tc_commit(done);
        }
        __syncwarp();
        const bool ok = tc::mbar_wait_warp(done, 0u, &abort_flag, &res->error, &res->error_info, kProbeMmaCode, kProbeLimit);
        asm volatile("mov.u64 %0, %%clock64;" : "=l"(t1)::"memory");
        if (blockIdx.x == 0 && lane == 0 && ok) {
            res->mma_cycles = (unsigned long long)(t1 - t0);
            res->mma_count = 8ull * kProbeChains;
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (mode == 0 && blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long longest = 0ull;
        bool all = true;
        for (int i = 0; i < kProbeWarps; ++i) { longest = max(longest, warp_cycles[i]); all = all && warp_cycles[i] != 0ull; }
        if (all) {
            res->copy_cycles = longest;
            res->copy_bytes = (unsigned long long)kProbeWarps * kProbeCopies * kProbeCopy;
        }
    }
    if (mode == 1 && warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc_512(tmem_slot);
    }
}

}  // namespace
}  // namespace stream

extern "C" size_t stream_probe_scratch_bytes(void) {
    const int n_sm = stream::tc::sm_count();
    return n_sm <= 0 ? 0 : 256 + (size_t)n_sm * stream::kProbeSlice * stream::kProbeCopy;
}

extern "C" stream_status stream_probe_unit_rates(void *scratch, size_t scratch_bytes, stream_unit_rates *out_host, void *cuda_stream) {
    using namespace stream;
    if (out_host == nullptr) { set_error("out_host must not be NULL"); return STREAM_ERR_INVALID_ARG; }
    const int n_sm = tc::sm_count();
    if (n_sm <= 0) { set_error("cannot read the SM count of the current device"); return STREAM_ERR_CUDA; }
    const size_t need = stream_probe_scratch_bytes();
    if (scratch == nullptr || scratch_bytes < need || ((uintptr_t)scratch & 255) != 0) {
        set_error("scratch must be a 256-byte aligned device buffer of at least %zu bytes", need);
        return STREAM_ERR_WORKSPACE;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemsetAsync(scratch, 0, need, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(scratch)");
    e = cudaFuncSetAttribute(probe_rates_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(probe)");
    ProbeResult *res = (ProbeResult *)scratch;
    const unsigned char *src = (const unsigned char *)scratch + 256;
    for (int mode = 0; mode < 2; ++mode) {
        probe_rates_kernel<<<n_sm, 64, kProbeSmem, st>>>(src, res, mode);
        e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "probe launch");
    }
    ProbeResult h;
    e = cudaMemcpyAsync(&h, res, sizeof(h), cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(probe result)");
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    out_host->tma_bytes_per_clk = h.copy_cycles ? (double)h.copy_bytes / (double)h.copy_cycles : 0.0;
    out_host->mma_cycles_m128n64 = h.mma_count ? (double)h.mma_cycles / (double)h.mma_count : 0.0;
    out_host->error = h.error;
    if (h.error != 0) {
        set_error("the probe kernel gave up on a bounded wait: code %u, info %u", h.error, h.error_info);
        return STREAM_ERR_DEVICE_CHECK;
    }
    return STREAM_OK;
}

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
