// Generic Stream mask kernel: one CTA per (batch, head, query block), fp32 FMA scoring.
// Covers every dtype / block size / head dim the ABI accepts; the tensor-core kernel takes the
// bf16, d = 128, 64x64 case. Follows Algorithm 2 with two exact shortcuts: only branches that
// contain an allowed block are kept in the candidate list (the others score -inf and can never
// displace a finite score), and a left branch inherits its parent's score (same representative).
#include <math_constants.h>

#include "common.cuh"

namespace stream {
namespace {

constexpr int kThreads = 256;
constexpr int kTile = 64;  // smem tiles hold up to 64 rows

// Masked maximum dot product (Eq. 4 under C) between the resident query tile and key block r.
// All threads must call; all get the result.
template <typename T, int D>
__device__ float tile_score(const Geom &g, const float *Qs, float *Ks, float *red, const T *kp, int qb, int r) {
    const int tid = threadIdx.x;
    __syncthreads();  // previous users of Ks / red are done
    for (int idx = tid; idx < kTile * D; idx += kThreads) {
        int n = idx / D, c = idx % D;
        long long tk = (long long)r * g.bk + n;
        Ks[n * (D + 1) + c] = (n < g.bk && tk < g.T) ? to_float(kp[tk * g.ks_t + c]) : 0.f;
    }
    __syncthreads();
    const int tx = tid % 16, ty = tid / 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 4
    for (int c = 0; c < D; ++c) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = Qs[(ty + 16 * i) * D + c];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Ks[(tx + 16 * j) * (D + 1) + c];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    float best = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int m = ty + 16 * i, n = tx + 16 * j;
            long long tq = (long long)qb * g.bq + m, tk = (long long)r * g.bk + n;
            bool ok = m < g.bq && n < g.bk && tq < g.T && tk < g.T && (!g.causal || tk <= tq);
            if (ok) best = fmaxf(best, acc[i][j]);
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
    if ((tid & 31) == 0) red[tid >> 5] = best;
    __syncthreads();
    float out = red[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) out = fmaxf(out, red[w]);
    return out;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) mask_generic_kernel(Geom g, MultiK mk, const T *__restrict__ q,
                                                                const T *__restrict__ k, int32_t *__restrict__ mask,
                                                                float *__restrict__ score, WorkspaceHeader *ws) {
    extern __shared__ float smem[];
    float *Qs = smem;                    // [64][D]
    float *Ks = Qs + kTile * D;          // [64][D + 1]
    float *node_s = Ks + kTile * (D + 1);  // [k]
    float *cand_s = node_s + g.k_top;    // [2k]
    int *node_f = (int *)(cand_s + 2 * g.k_top);  // [k]
    int *node_l = node_f + g.k_top;      // [k]
    int *cand_f = node_l + g.k_top;      // [2k]
    int *cand_l = cand_f + 2 * g.k_top;  // [2k]
    int *keep = cand_l + 2 * g.k_top;    // [2k]
    // several k: scores of this row by key block, NaN = not scored yet (a score does not depend on k)
    float *cache = mk.use_cache ? (float *)(keep + 2 * g.k_top) : nullptr;  // [N_k]
    __shared__ float red[kThreads / 32];
    __shared__ int s_nodes, s_cands;

    const int tid = threadIdx.x;
    // heaviest rows (late query blocks) first
    const long long row_rev = blockIdx.x;
    const int qb = g.n_qb - 1 - (int)(row_rev / ((long long)g.batch * g.H));
    const int bh = (int)(row_rev % ((long long)g.batch * g.H));
    const int b = bh / g.H, h = bh % g.H, kvh = h / g.hpg;
    const long long row = ((long long)b * g.H + h) * g.n_qb + qb;
    const T *qp = q + b * g.qs_b + h * g.qs_h;
    const T *kp = k + b * g.ks_b + kvh * g.ks_h;
    const int q_lim = last_valid_block(g, qb);
    const long long rows_total = (long long)g.batch * g.H * g.n_qb;

    if (cache != nullptr)
        for (int r = tid; r < g.N_k; r += kThreads) cache[r] = CUDART_NAN_F;
    for (int idx = tid; idx < kTile * D; idx += kThreads) {
        int m = idx / D, c = idx % D;
        long long tq = (long long)qb * g.bq + m;
        Qs[idx] = (m < g.bq && tq < g.T) ? to_float(qp[tq * g.qs_t + c]) : 0.f;
    }
    unsigned tiles = 0;
    const int n_pass = mk.n > 0 ? mk.n : 1;
    for (int pass = 0; pass < n_pass; ++pass) {
    const int kq = mk.n > 0 ? mk.k[pass] : row_k(g, qb);  // this pass's k (= k_top unless told otherwise)
    const int levels = row_levels(g, kq);
    __syncthreads();  // the previous pass is done with the node arrays
    if (tid == 0) {  // initial nodes tiling [0, N_k); keep those that hold an allowed block
        int n = 0;
        for (int j = 0; j < kq; ++j) {
            int f = (int)(((long long)j * g.N_k) / kq);
            int l = (int)(((long long)(j + 1) * g.N_k) / kq) - 1;
            if (f <= l && f <= q_lim) { node_f[n] = f; node_l[n] = l; node_s[n] = CUDART_NAN_F; ++n; }
        }
        s_nodes = n;
    }
    __syncthreads();

    for (int level = 0; level < levels; ++level) {
        if (tid == 0) {
            int n = 0;
            for (int i = 0; i < s_nodes; ++i) {
                int f = node_f[i], l = node_l[i], m = (f + l) / 2;
                cand_f[n] = f; cand_l[n] = m; cand_s[n] = node_s[i]; ++n;
                if (m + 1 <= l && m + 1 <= q_lim) { cand_f[n] = m + 1; cand_l[n] = l; cand_s[n] = CUDART_NAN_F; ++n; }
            }
            s_cands = n;
        }
        __syncthreads();
        const int n_cand = s_cands;
        for (int c = 0; c < n_cand; ++c) {
            if (isnan(cand_s[c])) {  // uniform: shared value
                const int r = cand_f[c];
                float s = cache != nullptr ? cache[r] : CUDART_NAN_F;  // (uniform too)
                if (isnan(s)) {
                    s = tile_score<T, D>(g, Qs, Ks, red, kp, qb, r);
                    ++tiles;
                }
                __syncthreads();
                if (tid == 0) {
                    cand_s[c] = s;
                    if (cache != nullptr) cache[r] = s;
                }
            }
        }
        __syncthreads();
        // top-k by rank: a candidate is beaten by a higher score, or an equal score at a lower index
        for (int c = tid; c < n_cand; c += kThreads) {
            int rank = 0;
            if (n_cand > kq) {
                float s = cand_s[c];
                for (int u = 0; u < n_cand; ++u) {
                    float su = cand_s[u];
                    rank += (su > s) || (su == s && u < c);
                }
            }
            keep[c] = rank < kq;
        }
        __syncthreads();
        if (tid == 0) {  // survivors stay in ascending block order
            int n = 0;
            for (int c = 0; c < n_cand; ++c)
                if (keep[c]) { node_f[n] = cand_f[c]; node_l[n] = cand_l[c]; node_s[n] = cand_s[c]; ++n; }
            s_nodes = n;
        }
        __syncthreads();
    }
    const int n_nodes = s_nodes;
    if (score != nullptr) {  // only reachable with zero levels: scores were never needed
        for (int i = 0; i < n_nodes; ++i) {
            if (isnan(node_s[i])) {
                const int r = node_f[i];
                float s = cache != nullptr ? cache[r] : CUDART_NAN_F;
                if (isnan(s)) s = tile_score<T, D>(g, Qs, Ks, red, kp, qb, r);
                __syncthreads();
                if (tid == 0) {
                    node_s[i] = s;
                    if (cache != nullptr) cache[r] = s;
                }
            }
        }
        __syncthreads();
    }
    const long long o = (pass * rows_total + row) * g.k_top;
    for (int j = tid; j < g.k_top; j += kThreads) {
        mask[o + j] = j < n_nodes ? node_f[j] : -1;
        if (score != nullptr) score[o + j] = j < n_nodes ? node_s[j] : -CUDART_INF_F;
    }
    }  // pass
    if (tid == 0) {
        atomicAdd(&ws->tiles_scored, (unsigned long long)tiles);
        atomicAdd(&ws->rows, 1ull);
        if (g.row_tiles != nullptr) g.row_tiles[row] = tiles;
    }
}

constexpr size_t kMaxDynamicSmem = 227 * 1024 - 1024;  // (the kernel has a few static words too)

template <typename T, int D>
stream_status launch(const Geom &g, MultiK mk, const T *q, const T *k, int32_t *mask, float *score, WorkspaceHeader *ws,
                     cudaStream_t st) {
    size_t smem = sizeof(float) * (kTile * D + kTile * (D + 1) + 3 * (size_t)g.k_top) + sizeof(int) * 8 * (size_t)g.k_top;
    mk.use_cache = mk.n > 1 && smem + sizeof(float) * (size_t)g.N_k <= kMaxDynamicSmem;
    if (mk.use_cache) smem += sizeof(float) * (size_t)g.N_k;
    auto kern = mask_generic_kernel<T, D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(mask_generic)");
    long long rows = (long long)g.batch * g.H * g.n_qb;
    kern<<<(unsigned)rows, kThreads, smem, st>>>(g, mk, q, k, mask, score, ws);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "mask_generic launch");
    return STREAM_OK;
}

template <typename T>
stream_status dispatch_d(const Geom &g, const MultiK &mk, const void *q, const void *k, int32_t *mask, float *score,
                         WorkspaceHeader *ws, cudaStream_t st) {
    const T *qq = (const T *)q, *kk = (const T *)k;
    switch (g.d) {
        case 16: return launch<T, 16>(g, mk, qq, kk, mask, score, ws, st);
        case 32: return launch<T, 32>(g, mk, qq, kk, mask, score, ws, st);
        case 64: return launch<T, 64>(g, mk, qq, kk, mask, score, ws, st);
        case 128: return launch<T, 128>(g, mk, qq, kk, mask, score, ws, st);
        case 256: return launch<T, 256>(g, mk, qq, kk, mask, score, ws, st);
    }
    set_error("generic mask kernel: head dim %d not in {16, 32, 64, 128, 256}", g.d);
    return STREAM_ERR_UNSUPPORTED;
}

}  // namespace

stream_status launch_mask_generic_multi(const Geom &g, const MultiK &mk, int dtype, const void *q, const void *k,
                                        int32_t *mask, float *score, WorkspaceHeader *ws, cudaStream_t st) {
    if (g.bq > kTile || g.bk > kTile) {
        set_error("generic mask kernel: block sizes up to %d (got %d, %d)", kTile, g.bq, g.bk);
        return STREAM_ERR_UNSUPPORTED;
    }
    if (dtype == STREAM_F32) return dispatch_d<float>(g, mk, q, k, mask, score, ws, st);
    return dispatch_d<__nv_bfloat16>(g, mk, q, k, mask, score, ws, st);
}

stream_status launch_mask_generic(const Geom &g, int dtype, const void *q, const void *k, int32_t *mask,
                                  float *score, WorkspaceHeader *ws, cudaStream_t st) {
    MultiK single = {};
    return launch_mask_generic_multi(g, single, dtype, q, k, mask, score, ws, st);
}

}  // namespace stream
