// Vertical attention scores of a Stream mask and their kurtosis (Section 4.1 of the paper: the
// column sums of the mask show which key blocks attract the later queries; heads whose vertical
// scores have a high kurtosis are the "receiver heads").
//
// Two kernels. The first spreads every head's mask rows over enough CTAs to fill the GPU: each
// CTA scans its rows coalesced (and, for the score-weighted form, the scores), adds them into a
// histogram over the key blocks in shared memory, and flushes the bins it touched into the output
// with global atomics. A lane always reads the same slot of the rows it meets (when k_top divides
// or is a multiple of 32), and the first slots name the same few blocks row after row (the sink
// block is kept by nearly every row): each lane therefore keeps the bin it met last and its sum in
// registers and only goes to the shared histogram when the bin changes, which takes the hot
// columns out of the atomics altogether. The second kernel, one CTA per head, reduces the head's
// vertical scores to their moments. A pure scan of the mask: bounded by HBM bandwidth.
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

// grid = (slices, heads); slice z of a head takes query blocks [z * rows_per, (z + 1) * rows_per).
__global__ void __launch_bounds__(kThreads) vertical_hist_kernel(int n_qb, int rows_per, int k_top, int n_kb,
                                                                  const int32_t *__restrict__ mask, const float *__restrict__ score,
                                                                  float *__restrict__ vertical, unsigned int *bad) {
    extern __shared__ float hist[];
    const long long head = blockIdx.y;
    for (int r = threadIdx.x; r < n_kb; r += kThreads) hist[r] = 0.f;
    __syncthreads();
    const int qb0 = blockIdx.x * rows_per, qb1 = min(n_qb, qb0 + rows_per);
    const long long first = ((long long)head * n_qb + qb0) * k_top, n = (long long)(qb1 - qb0) * k_top;
    const int32_t *m = mask + first;
    const float *s = score ? score + first : nullptr;
    int held = -1;      // the bin this lane met last
    float sum = 0.f;    // what it has gathered for it
    for (long long i = threadIdx.x; i < n; i += kThreads) {
        const int r = m[i];
        if (r < 0) continue;
        if (r >= n_kb) { atomicOr(bad, 1u); continue; }  // reported by the caller; never written out of range
        const float v = s ? s[i] : 1.f;
        if (r != held) {
            if (held >= 0) atomicAdd(&hist[held], sum);
            held = r;
            sum = 0.f;
        }
        sum += v;
    }
    if (held >= 0) atomicAdd(&hist[held], sum);
    __syncthreads();
    for (int r = threadIdx.x; r < n_kb; r += kThreads) {
        const float v = hist[r];
        if (v != 0.f) atomicAdd(&vertical[head * n_kb + r], v);
    }
}

// One CTA per head: Pearson kurtosis m4 / m2^2 of the head's vertical scores.
__global__ void __launch_bounds__(kThreads) vertical_moments_kernel(int n_kb, const float *__restrict__ vertical,
                                                                     float *__restrict__ kurtosis) {
    __shared__ float red[kThreads / 32];
    const float *v = vertical + (long long)blockIdx.x * n_kb;
    float part = 0.f;
    for (int r = threadIdx.x; r < n_kb; r += kThreads) part += v[r];
    const float mean = block_sum(part, red) / (float)n_kb;
    float p2 = 0.f, p4 = 0.f;
    for (int r = threadIdx.x; r < n_kb; r += kThreads) {
        const float d = v[r] - mean, d2 = d * d;
        p2 += d2;
        p4 += d2 * d2;
    }
    const float m2 = block_sum(p2, red) / (float)n_kb, m4 = block_sum(p4, red) / (float)n_kb;
    if (threadIdx.x == 0) kurtosis[blockIdx.x] = m2 > 0.f ? m4 / (m2 * m2) : 0.f;
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
    cudaError_t e = cudaFuncSetAttribute(vertical_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(vertical)");
    const int heads = g.batch * g.H;
    e = cudaMemsetAsync(vertical, 0, (size_t)heads * n_kb * sizeof(float), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(vertical)");
    // enough slices per head to give every SM a couple of CTAs, none shorter than 64 query blocks
    int n_sm = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n_sm = 148;
    int slices = (2 * n_sm + heads - 1) / heads;
    const int max_slices = (g.n_qb + 63) / 64;
    if (slices > max_slices) slices = max_slices;
    if (slices < 1) slices = 1;
    const int rows_per = (g.n_qb + slices - 1) / slices;
    slices = (g.n_qb + rows_per - 1) / rows_per;
    vertical_hist_kernel<<<dim3((unsigned)slices, (unsigned)heads), kThreads, smem, st>>>(g.n_qb, rows_per, g.k_top, (int)n_kb, mask,
                                                                                         score, vertical, bad_flag);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "vertical launch");
    if (kurtosis != nullptr) {
        vertical_moments_kernel<<<(unsigned)heads, kThreads, 0, st>>>((int)n_kb, vertical, kurtosis);
        e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "vertical moments launch");
    }
    return STREAM_OK;
}

}  // namespace stream
