// extern "C" boundary of libstream: argument validation, geometry, dispatch. See stream.h.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace stream {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

stream_status cuda_fail(cudaError_t e, const char *what) {
    set_error("%s: %s", what, cudaGetErrorString(e));
    return STREAM_ERR_CUDA;
}

namespace {

long long gcd_ll(long long a, long long b) {
    while (b) { long long t = a % b; a = b; b = t; }
    return a;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Validates *p and fills the kernel-side geometry.
stream_status make_geom(const stream_problem *p, Geom *g) {
    if (p == nullptr) { set_error("problem is NULL"); return STREAM_ERR_INVALID_ARG; }
    if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->n_q_heads % p->n_kv_heads != 0) {
        set_error("need batch >= 1 and n_kv_heads dividing n_q_heads (got %d, %d, %d)", p->batch, p->n_q_heads, p->n_kv_heads);
        return STREAM_ERR_INVALID_ARG;
    }
    if (p->T < 1 || p->d < 1 || p->block_q < 1 || p->block_k < 1 || p->k_top < 1) {
        set_error("T, d, block_q, block_k and k_top must be positive");
        return STREAM_ERR_INVALID_ARG;
    }
    if (p->dtype != STREAM_F32 && p->dtype != STREAM_BF16) { set_error("unknown dtype %d", p->dtype); return STREAM_ERR_INVALID_ARG; }
    if (p->impl < STREAM_IMPL_AUTO || p->impl > STREAM_IMPL_TENSOR) { set_error("unknown impl %d", p->impl); return STREAM_ERR_INVALID_ARG; }
    if (p->causal != 0 && p->causal != 1) { set_error("causal must be 0 or 1"); return STREAM_ERR_INVALID_ARG; }
    if (p->q_stride_t < p->d || p->kv_stride_t < p->d || p->q_stride_h < 0 || p->kv_stride_h < 0 || p->q_stride_b < 0 ||
        p->kv_stride_b < 0) {
        set_error("token strides must be >= d and head/batch strides non-negative");
        return STREAM_ERR_INVALID_ARG;
    }
    if (p->k_top > kMaxKTop) { set_error("k_top up to %d (got %d)", kMaxKTop, p->k_top); return STREAM_ERR_UNSUPPORTED; }
    long long lcm = (long long)p->block_q / gcd_ll(p->block_q, p->block_k) * p->block_k;
    long long Tp = (p->T + lcm - 1) / lcm * lcm;
    long long n_qb = (p->T + p->block_q - 1) / p->block_q, N_k = Tp / p->block_k;
    if (n_qb > 0x7fffffffLL || N_k > 0x7fffffffLL || (long long)p->batch * p->n_q_heads * n_qb > 0x7fffffffLL) {
        set_error("too many blocks or rows for 32-bit indexing");
        return STREAM_ERR_UNSUPPORTED;
    }
    g->batch = p->batch; g->H = p->n_q_heads; g->G = p->n_kv_heads; g->hpg = p->n_q_heads / p->n_kv_heads;
    g->T = p->T; g->d = p->d; g->bq = p->block_q; g->bk = p->block_k; g->k_top = p->k_top; g->causal = p->causal;
    g->n_qb = (int)n_qb; g->N_k = (int)N_k;
    g->levels = levels_for((int)N_k, p->k_top);
    g->k_row = nullptr;
    g->k_override = 0;
    g->row_tiles = nullptr;
    g->qs_b = p->q_stride_b; g->qs_h = p->q_stride_h; g->qs_t = p->q_stride_t;
    g->ks_b = p->kv_stride_b; g->ks_h = p->kv_stride_h; g->ks_t = p->kv_stride_t;
    return STREAM_OK;
}

size_t elem_size(int dtype) { return dtype == STREAM_F32 ? 4 : 2; }

struct StagingLayout { size_t q, k, v, mask, out, ws, k_row, total; };

StagingLayout staging_layout(const stream_problem *p, const Geom &g) {
    StagingLayout s;
    size_t e = elem_size(p->dtype);
    size_t qb = (size_t)g.batch * g.H * g.T * g.d * e, kb = (size_t)g.batch * g.G * g.T * g.d * e;
    size_t mb = (size_t)g.batch * g.H * g.n_qb * g.k_top * sizeof(int32_t);
    s.q = 0; s.k = s.q + align256(qb); s.v = s.k + align256(kb); s.mask = s.v + align256(kb);
    s.out = s.mask + align256(mb); s.ws = s.out + align256(qb);
    s.k_row = s.ws + sizeof(WorkspaceHeader);  // one k per query block, for the variable-k path
    s.total = s.k_row + align256((size_t)g.n_qb * sizeof(int32_t));
    return s;
}

// Streams and events behind stream_run_host, made once per device and kept for the life of the
// process: one stream for the copies in, one for the copies out (the kernels run on the
// caller's stream), and a few events to chain the three.
constexpr int kPipeEvents = 4;
struct HostPipe {
    bool ready = false;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, finish = nullptr, in_done[kPipeEvents] = {}, comp_done[kPipeEvents] = {};
};
constexpr int kMaxPipeDevices = 64;
std::mutex g_pipe_mu;
HostPipe g_pipes[kMaxPipeDevices];

stream_status host_pipe_for_current_device(HostPipe **out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxPipeDevices) { set_error("device ordinal %d outside 0..%d", dev, kMaxPipeDevices - 1); return STREAM_ERR_UNSUPPORTED; }
    std::lock_guard<std::mutex> lock(g_pipe_mu);
    HostPipe &hp = g_pipes[dev];
    if (!hp.ready) {
        if ((e = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e, "cudaStreamCreate");
        if ((e = cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e, "cudaStreamCreate");
        cudaEvent_t *evs[2 + 2 * kPipeEvents] = {&hp.start, &hp.finish};
        for (int i = 0; i < kPipeEvents; ++i) { evs[2 + i] = &hp.in_done[i]; evs[2 + kPipeEvents + i] = &hp.comp_done[i]; }
        for (cudaEvent_t *ev : evs)
            if ((e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e, "cudaEventCreate");
        hp.ready = true;
    }
    *out = &hp;
    return STREAM_OK;
}

bool dense_layout(const stream_problem *p) {
    return p->q_stride_t == p->d && p->q_stride_h == p->T * p->d && p->q_stride_b == (long long)p->n_q_heads * p->T * p->d &&
           p->kv_stride_t == p->d && p->kv_stride_h == p->T * p->d && p->kv_stride_b == (long long)p->n_kv_heads * p->T * p->d;
}

}  // namespace
}  // namespace stream

using namespace stream;

extern "C" {

int stream_version(void) { return 100; }

const char *stream_last_error(void) { return g_err; }

size_t stream_workspace_bytes(const stream_problem *p) {
    Geom g;
    if (make_geom(p, &g) != STREAM_OK) return 0;
    return sizeof(WorkspaceHeader);
}

// Both mask entry points: k_row == NULL is the fixed-k build.
static stream_status build_mask_impl(const stream_problem *p, const void *q, const void *k, const int32_t *k_row,
                                     int32_t *mask_out, float *score_out, void *workspace, size_t workspace_bytes,
                                     void *cuda_stream) {
    Geom g;
    stream_status rc = make_geom(p, &g);
    if (rc != STREAM_OK) return rc;
    g.k_row = k_row;
    if (q == nullptr || k == nullptr || mask_out == nullptr) { set_error("q, k and mask_out must not be NULL"); return STREAM_ERR_INVALID_ARG; }
    if (workspace == nullptr || workspace_bytes < sizeof(WorkspaceHeader) || ((uintptr_t)workspace & 255) != 0) {
        set_error("workspace must be a 256-byte aligned device buffer of at least %zu bytes", sizeof(WorkspaceHeader));
        return STREAM_ERR_WORKSPACE;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    WorkspaceHeader *ws = (WorkspaceHeader *)workspace;
    const bool tc_ok = mask_tc_supported(g, p->dtype), tok_ok = mask_tok_supported(g, p->dtype);
    if (p->impl == STREAM_IMPL_TENSOR && !tc_ok && !tok_ok) {
        set_error("tensor-core mask kernels need bf16, d = 128, block_k = 64, block_q = 64 or (with one k and at most 32768 key "
                  "blocks) 1, k_top <= 32, more than one key block, 16-byte aligned strides");
        return STREAM_ERR_UNSUPPORTED;
    }
    cudaError_t e = cudaMemsetAsync(ws, 0, sizeof(WorkspaceHeader), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(workspace)");
    // room behind the header for one counter per row: the build also says how many tiles each row scored
    const size_t n_rows = (size_t)g.batch * g.H * g.n_qb;
    if (workspace_bytes >= sizeof(WorkspaceHeader) + n_rows * sizeof(unsigned int)) g.row_tiles = (unsigned int *)(ws + 1);
    if (tc_ok && p->impl != STREAM_IMPL_GENERIC) return launch_mask_tc(g, q, k, mask_out, score_out, ws, st);
    if (tok_ok && p->impl != STREAM_IMPL_GENERIC) return launch_mask_tok(g, q, k, mask_out, score_out, ws, st);
    return launch_mask_generic(g, p->dtype, q, k, mask_out, score_out, ws, st);
}

size_t stream_workspace_bytes_multi(const stream_problem *p, int32_t n_k) {
    Geom g;
    if (make_geom(p, &g) != STREAM_OK) return 0;
    if (n_k < 1 || n_k > kMaxMultiK) { set_error("between 1 and %d sparsity constants per call (got %d)", kMaxMultiK, n_k); return 0; }
    size_t need = sizeof(WorkspaceHeader);
    if (n_k > 1 && p->impl != STREAM_IMPL_GENERIC && mask_tc_supported(g, p->dtype)) need += mask_tc_score_memory_bytes(g);
    return need;
}

stream_status stream_build_mask(const stream_problem *p, const void *q, const void *k, int32_t *mask_out,
                                float *score_out, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return build_mask_impl(p, q, k, nullptr, mask_out, score_out, workspace, workspace_bytes, cuda_stream);
}

stream_status stream_build_mask_var(const stream_problem *p, const void *q, const void *k, const int32_t *k_row,
                                    int32_t *mask_out, float *score_out, void *workspace, size_t workspace_bytes,
                                    void *cuda_stream) {
    if (k_row == nullptr) { set_error("k_row must not be NULL (use stream_build_mask for one k)"); return STREAM_ERR_INVALID_ARG; }
    return build_mask_impl(p, q, k, k_row, mask_out, score_out, workspace, workspace_bytes, cuda_stream);
}

stream_status stream_build_mask_multi(const stream_problem *p, const void *q, const void *k, int32_t n_k,
                                      const int32_t *k_list_host, int32_t *mask_out, float *score_out, void *workspace,
                                      size_t workspace_bytes, void *cuda_stream) {
    Geom g;
    stream_status rc = make_geom(p, &g);
    if (rc != STREAM_OK) return rc;
    if (q == nullptr || k == nullptr || mask_out == nullptr || k_list_host == nullptr) {
        set_error("q, k, k_list_host and mask_out must not be NULL");
        return STREAM_ERR_INVALID_ARG;
    }
    if (n_k < 1 || n_k > kMaxMultiK) { set_error("between 1 and %d sparsity constants per call (got %d)", kMaxMultiK, n_k); return STREAM_ERR_INVALID_ARG; }
    MultiK mk = {};
    mk.n = n_k;
    for (int i = 0; i < n_k; ++i) {
        if (k_list_host[i] < 1 || k_list_host[i] > g.k_top) {
            set_error("k_list_host[%d] = %d outside 1 .. k_top = %d", i, k_list_host[i], g.k_top);
            return STREAM_ERR_INVALID_ARG;
        }
        mk.k[i] = k_list_host[i];
    }
    if (workspace == nullptr || workspace_bytes < sizeof(WorkspaceHeader) || ((uintptr_t)workspace & 255) != 0) {
        set_error("workspace must be a 256-byte aligned device buffer of at least %zu bytes", sizeof(WorkspaceHeader));
        return STREAM_ERR_WORKSPACE;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    WorkspaceHeader *ws = (WorkspaceHeader *)workspace;
    const bool tc_ok = mask_tc_supported(g, p->dtype);
    if (p->impl == STREAM_IMPL_TENSOR && !tc_ok) {
        set_error("tensor-core mask kernel needs bf16, d = 128, block_q = block_k = 64, k_top <= 32, more than one key block, 16-byte aligned strides");
        return STREAM_ERR_UNSUPPORTED;
    }
    cudaError_t e = cudaMemsetAsync(ws, 0, sizeof(WorkspaceHeader), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(workspace)");
    if (!(tc_ok && p->impl != STREAM_IMPL_GENERIC))
        return launch_mask_generic_multi(g, mk, p->dtype, q, k, mask_out, score_out, ws, st);
    // tensor-core kernel, workspace large enough for its score memory: one launch walks every k of
    // a group before it moves on, and scores each (row, block) tile once
    const size_t score_bytes = mask_tc_score_memory_bytes(g);
    if (score_bytes > 0 && workspace_bytes >= sizeof(WorkspaceHeader) + score_bytes)
        return launch_mask_tc_multi(g, mk, q, k, mask_out, score_out, ws, (char *)workspace + sizeof(WorkspaceHeader), st);
    // otherwise one launch per k on the same stream (the counters add up; the work counter of the
    // persistent kernel starts again at 0 for each)
    const size_t per_k = (size_t)g.batch * g.H * g.n_qb * g.k_top;
    for (int i = 0; i < n_k; ++i) {
        if (i > 0) {
            e = cudaMemsetAsync(&ws->work_counter, 0, sizeof(ws->work_counter), st);
            if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(work counter)");
        }
        Geom gi = g;
        gi.k_override = mk.k[i];
        rc = launch_mask_tc(gi, q, k, mask_out + i * per_k, score_out != nullptr ? score_out + i * per_k : nullptr, ws, st);
        if (rc != STREAM_OK) return rc;
    }
    return STREAM_OK;
}

stream_status stream_k_schedule(const stream_problem *p, double s, int32_t *k_row_host) {
    Geom g;
    stream_status rc = make_geom(p, &g);
    if (rc != STREAM_OK) return rc;
    if (k_row_host == nullptr) { set_error("k_row_host must not be NULL"); return STREAM_ERR_INVALID_ARG; }
    if (!(s > 0.0 && s < 1.0)) { set_error("effective sparsity must lie strictly between 0 and 1 (got %g)", s); return STREAM_ERR_INVALID_ARG; }
    for (int qb = 0; qb < g.n_qb; ++qb) {
        const long long n = (long long)last_valid_block(g, qb) + 1;  // key blocks the row may look at
        long long kq = (long long)floor(1.0 + (double)(n - 1) * s);
        k_row_host[qb] = (int32_t)(kq < 1 ? 1 : (kq > g.k_top ? g.k_top : kq));
    }
    return STREAM_OK;
}

stream_status stream_effective_k(int64_t T, int32_t block_q, double s, int32_t *k_out_host) {
    if (k_out_host == nullptr) { set_error("k_out_host must not be NULL"); return STREAM_ERR_INVALID_ARG; }
    if (T < 1 || block_q < 1) { set_error("T and block_q must be positive"); return STREAM_ERR_INVALID_ARG; }
    if (!(s >= 0.0 && s <= 1.0)) { set_error("effective sparsity must lie in [0, 1] (got %g)", s); return STREAM_ERR_INVALID_ARG; }
    const double n = (double)T / (double)block_q;            // T / b_q as the formula has it (not rounded)
    const long long n_rows = T / block_q > 1 ? T / block_q : 1;  // floor(T / b_q), the upper end of k's range
    long long kq = (long long)floor(1.0 + (n - 1.0) * s);
    kq = kq < 1 ? 1 : (kq > n_rows ? n_rows : kq);
    if (kq > 0x7fffffffLL) { set_error("k does not fit 32 bits"); return STREAM_ERR_UNSUPPORTED; }
    *k_out_host = (int32_t)kq;
    return STREAM_OK;
}

stream_status stream_sparse_attention(const stream_problem *p, const void *q, const void *k, const void *v,
                                      const int32_t *mask, float scale, void *out, void *cuda_stream) {
    Geom g;
    stream_status rc = make_geom(p, &g);
    if (rc != STREAM_OK) return rc;
    if (q == nullptr || k == nullptr || v == nullptr || mask == nullptr || out == nullptr) {
        set_error("q, k, v, mask and out must not be NULL");
        return STREAM_ERR_INVALID_ARG;
    }
    if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)g.d);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const bool tc_ok = attn_tc_supported(g, p->dtype);
    if (p->impl == STREAM_IMPL_TENSOR && !tc_ok) {
        set_error("tensor-core attention kernel needs bf16, d = 128, block_q = block_k = 64, 16-byte aligned strides");
        return STREAM_ERR_UNSUPPORTED;
    }
    if (tc_ok && p->impl != STREAM_IMPL_GENERIC) return launch_attn_tc(g, q, k, v, mask, scale, out, st);
    return launch_attn_generic(g, p->dtype, q, k, v, mask, scale, out, st);
}

stream_status stream_read_stats(const void *workspace, stream_stats *out, void *cuda_stream) {
    if (workspace == nullptr || out == nullptr) { set_error("workspace and out must not be NULL"); return STREAM_ERR_INVALID_ARG; }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemcpyAsync(out, workspace, sizeof(stream_stats), cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(stats)");
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    if (out->error != 0) {
        set_error("a kernel recorded a failed device-side check: code %u, info %u", out->error, out->error_info);
        return STREAM_ERR_DEVICE_CHECK;
    }
    return STREAM_OK;
}

stream_status stream_vertical_scores(const stream_problem *p, const int32_t *mask, const float *scores, float *vertical_out,
                                     float *kurtosis_out, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    Geom g;
    stream_status rc = make_geom(p, &g);
    if (rc != STREAM_OK) return rc;
    if (mask == nullptr || vertical_out == nullptr) { set_error("mask and vertical_out must not be NULL"); return STREAM_ERR_INVALID_ARG; }
    if (workspace == nullptr || workspace_bytes < sizeof(WorkspaceHeader) || ((uintptr_t)workspace & 255) != 0) {
        set_error("workspace must be a 256-byte aligned device buffer of at least %zu bytes", sizeof(WorkspaceHeader));
        return STREAM_ERR_WORKSPACE;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    WorkspaceHeader *ws = (WorkspaceHeader *)workspace;
    cudaError_t e = cudaMemsetAsync(ws, 0, sizeof(WorkspaceHeader), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(workspace)");
    return launch_vertical(g, mask, scores, vertical_out, kurtosis_out, &ws->error, st);
}

stream_status stream_mask_difference(int64_t n_rows, int32_t k_a, const int32_t *mask_a, const float *scores_a, int32_t k_b,
                                     const int32_t *mask_b, int32_t *diff_out, float *diff_scores_out, void *cuda_stream) {
    if (n_rows < 0 || k_a < 1 || k_b < 1 || k_a > kMaxKTop || k_b > kMaxKTop) {
        set_error("need n_rows >= 0 and 1 <= k_a, k_b <= %d", kMaxKTop);
        return STREAM_ERR_INVALID_ARG;
    }
    if (mask_a == nullptr || mask_b == nullptr || diff_out == nullptr) { set_error("mask_a, mask_b and diff_out must not be NULL"); return STREAM_ERR_INVALID_ARG; }
    if (diff_scores_out != nullptr && scores_a == nullptr) { set_error("diff_scores_out needs scores_a"); return STREAM_ERR_INVALID_ARG; }
    return launch_mask_diff(n_rows, k_a, mask_a, scores_a, k_b, mask_b, diff_out, diff_scores_out, (cudaStream_t)cuda_stream);
}

stream_status stream_check_device_status(void *cuda_stream) {
    unsigned int words[2] = {0, 0};
    stream_status rc = read_attn_status(words, (cudaStream_t)cuda_stream);
    if (rc != STREAM_OK) return rc;
    if (words[0] != 0) {
        set_error("attention kernel gave up on a bounded wait: code %u, block %u", words[0], words[1]);
        return STREAM_ERR_DEVICE_CHECK;
    }
    return STREAM_OK;
}

size_t stream_host_staging_bytes(const stream_problem *p) {
    Geom g;
    if (make_geom(p, &g) != STREAM_OK) return 0;
    return staging_layout(p, g).total;
}

// Both host entry points: k_row_host == NULL is the fixed-k path.
static stream_status run_host_impl(const stream_problem *p, const void *q_host, const void *k_host, const void *v_host,
                                   const int32_t *k_row_host, int32_t *mask_host, void *out_host, float scale, void *staging,
                                   size_t staging_bytes, void *cuda_stream) {
    Geom g;
    stream_status rc = make_geom(p, &g);
    if (rc != STREAM_OK) return rc;
    if (!q_host || !k_host || !v_host || !mask_host || !out_host) { set_error("host pointers must not be NULL"); return STREAM_ERR_INVALID_ARG; }
    if (!dense_layout(p)) { set_error("stream_run_host needs dense [batch, heads, T, d] host tensors"); return STREAM_ERR_INVALID_ARG; }
    StagingLayout s = staging_layout(p, g);
    if (staging == nullptr || staging_bytes < s.total || ((uintptr_t)staging & 255) != 0) {
        set_error("staging must be a 256-byte aligned device buffer of at least %zu bytes", s.total);
        return STREAM_ERR_WORKSPACE;
    }
    HostPipe *hp = nullptr;
    rc = host_pipe_for_current_device(&hp);
    if (rc != STREAM_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char *base = (char *)staging;
    const size_t e = elem_size(p->dtype);
    // One chunk = one kv head of one batch entry with its query heads: nothing else depends on it,
    // so its copy in, its two kernels and its copy out can overlap with the neighbours'.
    const size_t q_chunk = (size_t)g.hpg * g.T * g.d * e, kv_chunk = (size_t)g.T * g.d * e;
    const size_t m_chunk = (size_t)g.hpg * g.n_qb * g.k_top * sizeof(int32_t);
    stream_problem sub = *p;
    sub.batch = 1; sub.n_q_heads = g.hpg; sub.n_kv_heads = 1;
    cudaError_t ce;
#define STREAM_TRY(call, what) do { if ((ce = (call)) != cudaSuccess) return cuda_fail(ce, what); } while (0)
    // the internal streams start after everything already enqueued on the caller's stream
    STREAM_TRY(cudaEventRecord(hp->start, st), "cudaEventRecord");
    STREAM_TRY(cudaStreamWaitEvent(hp->in, hp->start, 0), "cudaStreamWaitEvent");
    STREAM_TRY(cudaStreamWaitEvent(hp->out, hp->start, 0), "cudaStreamWaitEvent");
    const int32_t *k_row_dev = nullptr;
    if (k_row_host != nullptr) {  // ahead of the first chunk on the same stream: in place before its kernels wait on it
        STREAM_TRY(cudaMemcpyAsync(base + s.k_row, k_row_host, (size_t)g.n_qb * sizeof(int32_t), cudaMemcpyHostToDevice, hp->in), "H2D k_row");
        k_row_dev = (const int32_t *)(base + s.k_row);
    }
    const int n_chunks = g.batch * g.G;
    const size_t q_head = (size_t)g.T * g.d * e, m_head = (size_t)g.n_qb * g.k_top * sizeof(int32_t);
    int unit = 0;  // running number of the (chunk, heads) units, for the ring of events
    for (int c = 0; c < n_chunks; ++c) {
        const size_t ko = (size_t)c * kv_chunk;
        // The very last chunk goes through in two halves of its query heads: what is left after the
        // last byte has arrived (its kernels and its copy out, which nothing overlaps any more) is
        // then half as long. Everywhere else a chunk keeps all its heads together, so that the
        // first level's key tiles serve as many rows as possible.
        const int n_units = (c == n_chunks - 1 && g.hpg >= 4) ? 2 : 1;
        for (int u = 0; u < n_units; ++u, ++unit) {
            const int h0 = u * ((g.hpg + n_units - 1) / n_units);
            const int nh = (u == n_units - 1) ? g.hpg - h0 : (g.hpg + n_units - 1) / n_units;
            const size_t qo = (size_t)c * q_chunk + (size_t)h0 * q_head, mo = (size_t)c * m_chunk + (size_t)h0 * m_head;
            const size_t q_bytes = (size_t)nh * q_head, m_bytes = (size_t)nh * m_head;
            sub.n_q_heads = nh;
            cudaEvent_t in_done = hp->in_done[unit % kPipeEvents], comp_done = hp->comp_done[unit % kPipeEvents];
            if (u == 0) {
                STREAM_TRY(cudaMemcpyAsync(base + s.k + ko, (const char *)k_host + ko, kv_chunk, cudaMemcpyHostToDevice, hp->in), "H2D k");
                STREAM_TRY(cudaMemcpyAsync(base + s.v + ko, (const char *)v_host + ko, kv_chunk, cudaMemcpyHostToDevice, hp->in), "H2D v");
            }
            STREAM_TRY(cudaMemcpyAsync(base + s.q + qo, (const char *)q_host + qo, q_bytes, cudaMemcpyHostToDevice, hp->in), "H2D q");
            STREAM_TRY(cudaEventRecord(in_done, hp->in), "cudaEventRecord");
            STREAM_TRY(cudaStreamWaitEvent(st, in_done, 0), "cudaStreamWaitEvent");
            rc = build_mask_impl(&sub, base + s.q + qo, base + s.k + ko, k_row_dev, (int32_t *)(base + s.mask + mo), nullptr,
                                 base + s.ws, sizeof(WorkspaceHeader), cuda_stream);
            if (rc != STREAM_OK) return rc;
            rc = stream_sparse_attention(&sub, base + s.q + qo, base + s.k + ko, base + s.v + ko,
                                         (const int32_t *)(base + s.mask + mo), scale, base + s.out + qo, cuda_stream);
            if (rc != STREAM_OK) return rc;
            STREAM_TRY(cudaEventRecord(comp_done, st), "cudaEventRecord");
            STREAM_TRY(cudaStreamWaitEvent(hp->out, comp_done, 0), "cudaStreamWaitEvent");
            STREAM_TRY(cudaMemcpyAsync((char *)mask_host + mo, base + s.mask + mo, m_bytes, cudaMemcpyDeviceToHost, hp->out), "D2H mask");
            STREAM_TRY(cudaMemcpyAsync((char *)out_host + qo, base + s.out + qo, q_bytes, cudaMemcpyDeviceToHost, hp->out), "D2H out");
        }
    }
    // the caller's stream is done when the last copy out is
    STREAM_TRY(cudaEventRecord(hp->finish, hp->out), "cudaEventRecord");
    STREAM_TRY(cudaStreamWaitEvent(st, hp->finish, 0), "cudaStreamWaitEvent");
#undef STREAM_TRY
    return STREAM_OK;
}

stream_status stream_run_host(const stream_problem *p, const void *q_host, const void *k_host, const void *v_host,
                              int32_t *mask_host, void *out_host, float scale, void *staging,
                              size_t staging_bytes, void *cuda_stream) {
    return run_host_impl(p, q_host, k_host, v_host, nullptr, mask_host, out_host, scale, staging, staging_bytes, cuda_stream);
}

stream_status stream_run_host_var(const stream_problem *p, const void *q_host, const void *k_host, const void *v_host,
                                  const int32_t *k_row_host, int32_t *mask_host, void *out_host, float scale, void *staging,
                                  size_t staging_bytes, void *cuda_stream) {
    if (k_row_host == nullptr) { set_error("k_row_host must not be NULL (use stream_run_host for one k)"); return STREAM_ERR_INVALID_ARG; }
    return run_host_impl(p, q_host, k_host, v_host, k_row_host, mask_host, out_host, scale, staging, staging_bytes, cuda_stream);
}

}  // extern "C"
