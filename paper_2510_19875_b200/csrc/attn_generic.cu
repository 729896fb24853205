// Generic block-sparse attention (Eq. 2 on a Stream mask): one CTA per (batch, head, query
// block), fp32 FMA, online softmax over the kept key blocks. Covers every dtype / block size /
// head dim the ABI accepts.
#include <math_constants.h>

#include "common.cuh"

namespace stream {
namespace {

constexpr int kThreads = 256;
constexpr int kTile = 64;

template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ float from_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) attn_generic_kernel(Geom g, const T *__restrict__ q,
                                                                const T *__restrict__ k, const T *__restrict__ v,
                                                                const int32_t *__restrict__ mask, float scale,
                                                                T *__restrict__ out) {
    extern __shared__ float smem[];
    float *Qs = smem;                     // [64][D]
    float *Ks = Qs + kTile * D;           // [64][D + 1]
    float *Vs = Ks + kTile * (D + 1);     // [64][D]
    float *Ps = Vs + kTile * D;           // [64][65]

    const int tid = threadIdx.x;
    const long long row = blockIdx.x;
    const int qb = (int)(row % g.n_qb);
    const int bh = (int)(row / g.n_qb);
    const int b = bh / g.H, h = bh % g.H, kvh = h / g.hpg;
    const T *qp = q + b * g.qs_b + h * g.qs_h;
    const T *kp = k + b * g.ks_b + kvh * g.ks_h;
    const T *vp = v + b * g.ks_b + kvh * g.ks_h;
    const int32_t *mrow = mask + row * g.k_top;

    for (int idx = tid; idx < kTile * D; idx += kThreads) {
        int m = idx / D, c = idx % D;
        long long tq = (long long)qb * g.bq + m;
        Qs[idx] = (m < g.bq && tq < g.T) ? to_float(qp[tq * g.qs_t + c]) : 0.f;
    }
    const int tx = tid % 16, ty = tid / 16;  // logits: rows ty + 16 i, keys tx + 16 j
    const int om = tid / 4, og = tid % 4;    // output: row om, channels og + 4 i
    float o[D / 4];
#pragma unroll
    for (int i = 0; i < D / 4; ++i) o[i] = 0.f;
    float run_max = -CUDART_INF_F, run_sum = 0.f;

    for (int j = 0; j < g.k_top; ++j) {
        const int r = mrow[j];
        if (r < 0) continue;  // uniform: same value for the whole CTA
        __syncthreads();
        for (int idx = tid; idx < kTile * D; idx += kThreads) {
            int n = idx / D, c = idx % D;
            long long tk = (long long)r * g.bk + n;
            bool in = n < g.bk && tk < g.T;
            Ks[n * (D + 1) + c] = in ? to_float(kp[tk * g.ks_t + c]) : 0.f;
            Vs[idx] = in ? to_float(vp[tk * g.ks_t + c]) : 0.f;
        }
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) acc[i][jj] = 0.f;
#pragma unroll 4
        for (int c = 0; c < D; ++c) {
            float a[4], bb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = Qs[(ty + 16 * i) * D + c];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) bb[jj] = Ks[(tx + 16 * jj) * (D + 1) + c];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) acc[i][jj] = fmaf(a[i], bb[jj], acc[i][jj]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                int m = ty + 16 * i, n = tx + 16 * jj;
                long long tq = (long long)qb * g.bq + m, tk = (long long)r * g.bk + n;
                bool ok = m < g.bq && n < g.bk && tq < g.T && tk < g.T && (!g.causal || tk <= tq);
                Ps[m * (kTile + 1) + n] = ok ? scale * acc[i][jj] : -CUDART_INF_F;
            }
        __syncthreads();
        // online softmax: the four threads of a row split its keys
        float mx = -CUDART_INF_F;
        for (int n = og; n < kTile; n += 4) mx = fmaxf(mx, Ps[om * (kTile + 1) + n]);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float new_max = fmaxf(run_max, mx);
        const float alpha = (new_max == -CUDART_INF_F) ? 1.f : expf(run_max - new_max);
        float part = 0.f;
        for (int n = og; n < kTile; n += 4) {
            float s = Ps[om * (kTile + 1) + n];
            float p = (s == -CUDART_INF_F) ? 0.f : expf(s - new_max);
            Ps[om * (kTile + 1) + n] = p;
            part += p;
        }
        part += __shfl_xor_sync(0xffffffffu, part, 1);
        part += __shfl_xor_sync(0xffffffffu, part, 2);
        run_sum = run_sum * alpha + part;
        run_max = new_max;
        __syncwarp();
#pragma unroll
        for (int i = 0; i < D / 4; ++i) o[i] *= alpha;
        for (int n = 0; n < kTile; ++n) {
            float p = Ps[om * (kTile + 1) + n];
#pragma unroll
            for (int i = 0; i < D / 4; ++i) o[i] = fmaf(p, Vs[n * D + og + 4 * i], o[i]);
        }
    }
    const long long tq = (long long)qb * g.bq + om;
    if (om < g.bq && tq < g.T) {
        const float inv = run_sum > 0.f ? 1.f / run_sum : 0.f;
        T *op = out + (((long long)b * g.H + h) * g.T + tq) * D;
#pragma unroll
        for (int i = 0; i < D / 4; ++i) op[og + 4 * i] = from_float<T>(o[i] * inv);
    }
}

template <typename T, int D>
stream_status launch(const Geom &g, const T *q, const T *k, const T *v, const int32_t *mask, float scale, T *out,
                     cudaStream_t st) {
    size_t smem = sizeof(float) * (kTile * D * 2 + kTile * (D + 1) + kTile * (kTile + 1));
    auto kern = attn_generic_kernel<T, D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(attn_generic)");
    long long rows = (long long)g.batch * g.H * g.n_qb;
    kern<<<(unsigned)rows, kThreads, smem, st>>>(g, q, k, v, mask, scale, out);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "attn_generic launch");
    return STREAM_OK;
}

template <typename T>
stream_status dispatch_d(const Geom &g, const void *q, const void *k, const void *v, const int32_t *mask,
                         float scale, void *out, cudaStream_t st) {
    const T *qq = (const T *)q, *kk = (const T *)k, *vv = (const T *)v;
    switch (g.d) {
        case 16: return launch<T, 16>(g, qq, kk, vv, mask, scale, (T *)out, st);
        case 32: return launch<T, 32>(g, qq, kk, vv, mask, scale, (T *)out, st);
        case 64: return launch<T, 64>(g, qq, kk, vv, mask, scale, (T *)out, st);
        case 128: return launch<T, 128>(g, qq, kk, vv, mask, scale, (T *)out, st);
        case 256: return launch<T, 256>(g, qq, kk, vv, mask, scale, (T *)out, st);
    }
    set_error("generic attention kernel: head dim %d not in {16, 32, 64, 128, 256}", g.d);
    return STREAM_ERR_UNSUPPORTED;
}

}  // namespace

stream_status launch_attn_generic(const Geom &g, int dtype, const void *q, const void *k, const void *v,
                                  const int32_t *mask, float scale, void *out, cudaStream_t st) {
    if (g.bq > kTile || g.bk > kTile) {
        set_error("generic attention kernel: block sizes up to %d (got %d, %d)", kTile, g.bq, g.bk);
        return STREAM_ERR_UNSUPPORTED;
    }
    if (dtype == STREAM_F32) return dispatch_d<float>(g, q, k, v, mask, scale, out, st);
    return dispatch_d<__nv_bfloat16>(g, q, k, v, mask, scale, out, st);
}

}  // namespace stream
