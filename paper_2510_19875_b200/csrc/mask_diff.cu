// Mask subtraction (Section 4.2 of the paper, "Exploring Information Flow": the masks of a smaller
// budget k are subtracted from those of a larger one; what is left, weighted by the larger
// mask's block scores, are the connections only the larger budget keeps).
//
// One warp per row: every lane tests entries of row a against row b (held in registers, 32 at a
// time, compared through shuffles), and the survivors are compacted in order with ballots. A scan
// of the two masks: bounded by HBM bandwidth.
#include <math_constants.h>

#include "common.cuh"

namespace stream {
namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads) mask_diff_kernel(long long n_rows, int k_a, const int32_t *__restrict__ mask_a,
                                                             const float *__restrict__ score_a, int k_b,
                                                             const int32_t *__restrict__ mask_b, int32_t *__restrict__ diff,
                                                             float *__restrict__ diff_score) {
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (row >= n_rows) return;  // whole warps leave together
    const int32_t *a = mask_a + row * k_a, *b = mask_b + row * k_b;
    int n_out = 0;
    for (int j0 = 0; j0 < k_a; j0 += 32) {
        const int j = j0 + lane;
        const int va = j < k_a ? a[j] : -1;
        bool keep = va >= 0;
        for (int u0 = 0; u0 < k_b; u0 += 32) {
            const int vb = u0 + lane < k_b ? b[u0 + lane] : -1;
#pragma unroll 8
            for (int u = 0; u < 32; ++u) {
                const int other = __shfl_sync(0xffffffffu, vb, u);  // every lane takes part, whatever its own keep
                keep = keep & (other != va);
            }
        }
        const unsigned kept = __ballot_sync(0xffffffffu, keep);
        if (keep) {
            const int pos = n_out + __popc(kept & ((1u << lane) - 1u));
            diff[row * k_a + pos] = va;
            if (diff_score != nullptr) diff_score[row * k_a + pos] = score_a[row * k_a + j];
        }
        n_out += __popc(kept);
    }
    for (int pos = n_out + lane; pos < k_a; pos += 32) {
        diff[row * k_a + pos] = -1;
        if (diff_score != nullptr) diff_score[row * k_a + pos] = -CUDART_INF_F;
    }
}

}  // namespace

stream_status launch_mask_diff(long long n_rows, int k_a, const int32_t *mask_a, const float *score_a, int k_b,
                               const int32_t *mask_b, int32_t *diff, float *diff_score, cudaStream_t st) {
    if (n_rows == 0) return STREAM_OK;
    const long long blocks = (n_rows + kThreads / 32 - 1) / (kThreads / 32);
    if (blocks > 0x7fffffffLL) { set_error("too many rows for one launch"); return STREAM_ERR_UNSUPPORTED; }
    mask_diff_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(n_rows, k_a, mask_a, score_a, k_b, mask_b, diff, diff_score);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "mask_diff launch");
    return STREAM_OK;
}

}  // namespace stream
