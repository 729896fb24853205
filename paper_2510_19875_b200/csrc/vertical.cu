// Vertical attention scores of a Stream mask and their kurtosis (Section 4.1 of the paper: the
// column sums of the mask show which key blocks attract the later queries; heads whose vertical
// scores have a high kurtosis are the "receiver heads").
//
// One CTA per (batch, head): a histogram over the key blocks in shared memory, filled by a
// coalesced scan of the head's mask rows (and, for the score-weighted form, of the scores), then
// written out and reduced to the moments. A pure scan of the mask: bounded by HBM bandwidth.
#include "common.cuh"

namespace stream {
namespace {

constexpr int kThreads = 512;
constexpr int kMaxBins = 49152;  // key blocks per head that fit the shared-memory histogram

__device__ float block_sum(float x, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    __syncthreads();  // previous users of red are done
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    float s = 0.f;
    for (int w = 0; w < kThreads / 32; ++w) s += red[w];  // same order in every thread
    return s;
}

__global__ void __launch_bounds__(kThreads) vertical_kernel(int n_qb, int k_top, int n_kb, const int32_t *__restrict__ mask,
                                                             const float *__restrict__ score, float *__restrict__ vertical,
                                                             float *__restrict__ kurtosis, unsigned int *bad) {
    extern __shared__ float hist[];
    __shared__ float red[kThreads / 32];
    const long long head = blockIdx.x;
    for (int r = threadIdx.x; r < n_kb; r += kThreads) hist[r] = 0.f;
    __syncthreads();
    const long long n = (long long)n_qb * k_top;
    const int32_t *m = mask + head * n;
    const float *s = score ? score + head * n : nullptr;
    for (long long i = threadIdx.x; i < n; i += kThreads) {
        const int r = m[i];
        if (r < 0) continue;
        if (r >= n_kb) { atomicOr(bad, 1u); continue; }  // reported by the caller; never written out of range
        atomicAdd(&hist[r], s ? s[i] : 1.f);
    }
    __syncthreads();
    float part = 0.f;
    for (int r = threadIdx.x; r < n_kb; r += kThreads) {
        const float v = hist[r];
        vertical[head * n_kb + r] = v;
        part += v;
    }
    if (kurtosis == nullptr) return;
    const float mean = block_sum(part, red) / (float)n_kb;
    float p2 = 0.f, p4 = 0.f;
    for (int r = threadIdx.x; r < n_kb; r += kThreads) {
        const float d = hist[r] - mean, d2 = d * d;
        p2 += d2;
        p4 += d2 * d2;
    }
    const float m2 = block_sum(p2, red) / (float)n_kb, m4 = block_sum(p4, red) / (float)n_kb;
    if (threadIdx.x == 0) kurtosis[head] = m2 > 0.f ? m4 / (m2 * m2) : 0.f;
}

}  // namespace

stream_status launch_vertical(const Geom &g, const int32_t *mask, const float *score, float *vertical, float *kurtosis,
                              unsigned int *bad_flag, cudaStream_t st) {
    const long long n_kb = (g.T + g.bk - 1) / g.bk;
    if (n_kb > kMaxBins) {
        set_error("vertical scores: %lld key blocks per head, the kernel holds up to %d", n_kb, kMaxBins);
        return STREAM_ERR_UNSUPPORTED;
    }
    const size_t smem = (size_t)n_kb * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(vertical_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(vertical)");
    vertical_kernel<<<(unsigned)(g.batch * g.H), kThreads, smem, st>>>(g.n_qb, g.k_top, (int)n_kb, mask, score, vertical,
                                                                      kurtosis, bad_flag);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "vertical launch");
    return STREAM_OK;
}

}  // namespace stream
