// Shared declarations of the CUDA side of libstream (not shared with the CPU oracle).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "stream.h"

namespace stream {

// Problem geometry as the kernels see it.
struct Geom {
    int batch, H, G, hpg;       // heads; hpg = H / G
    long long T;
    int d, bq, bk, k_top, causal;
    int n_qb;                   // ceil(T / bq): rows per head
    int N_k;                    // key blocks after padding T to a multiple of lcm(bq, bk)
    int levels;                 // split levels that can change the result (with k = k_top)
    const int32_t *k_row;       // device, [n_qb]: k of each query block (clamped to 1 .. k_top), or NULL = k_top everywhere
    int k_override;             // > 0: every row uses this k (one launch of a several-k build); rows stay k_top wide
    unsigned int *row_tiles;    // device, [batch * H * n_qb] or NULL: tiles scored for each row (single-k builds)
    long long qs_b, qs_h, qs_t; // element strides
    long long ks_b, ks_h, ks_t;
};

// Header at the start of the mask workspace. The first 40 bytes mirror stream_stats.
struct WorkspaceHeader {
    unsigned long long tiles_scored;
    unsigned long long rows;
    unsigned int error;
    unsigned int error_info;
    unsigned long long tile_products;  // 64 x 64 tile products computed (more than tiles_scored where rows share a product)
    unsigned long long tiles_fetched;  // tiles copied into shared memory (the tensor-core block kernel counts them)
    unsigned int work_counter;  // next work item of the persistent kernels
    unsigned int pad[53];
};
static_assert(sizeof(WorkspaceHeader) == 256, "workspace header is 256 bytes");

constexpr int kMaxKTop = 1024;

// Several sparsity constants in one call.
constexpr int kMaxMultiK = 8;
struct MultiK {
    int n;               // 0: a single build (k from the geometry)
    int k[kMaxMultiK];
    int use_cache;       // generic kernel: N_k scores of the row fit in shared memory behind the tiles
};

void set_error(const char *fmt, ...);
stream_status cuda_fail(cudaError_t e, const char *what);

// Launchers (each validates what only it can support and returns UNSUPPORTED otherwise).
stream_status launch_mask_generic(const Geom &g, int dtype, const void *q, const void *k, int32_t *mask,
                                  float *score, WorkspaceHeader *ws, cudaStream_t st);
// mask / score: [mk.n][rows][k_top]; a row's tiles are scored once for all k where the cache fits.
stream_status launch_mask_generic_multi(const Geom &g, const MultiK &mk, int dtype, const void *q, const void *k,
                                        int32_t *mask, float *score, WorkspaceHeader *ws, cudaStream_t st);
stream_status launch_attn_generic(const Geom &g, int dtype, const void *q, const void *k, const void *v,
                                  const int32_t *mask, float scale, void *out, cudaStream_t st);
bool mask_tc_supported(const Geom &g, int dtype);
stream_status launch_mask_tc(const Geom &g, const void *q, const void *k, int32_t *mask, float *score,
                             WorkspaceHeader *ws, cudaStream_t st);
// Several k in one launch (mk.n >= 1: mask / score are [mk.n][rows][k_top]); with score_memory
// (mask_tc_score_memory_bytes(g) bytes, device) a (row, block) tile is scored once for all k.
size_t mask_tc_score_memory_bytes(const Geom &g);
stream_status launch_mask_tc_multi(const Geom &g, const MultiK &mk, const void *q, const void *k, int32_t *mask,
                                   float *score, WorkspaceHeader *ws, void *score_memory, cudaStream_t st);
// Per-token masks (block_q = 1) on the tensor cores.
bool mask_tok_supported(const Geom &g, int dtype);
stream_status launch_mask_tok(const Geom &g, const void *q, const void *k, int32_t *mask, float *score,
                              WorkspaceHeader *ws, cudaStream_t st);
bool attn_tc_supported(const Geom &g, int dtype);
stream_status launch_attn_tc(const Geom &g, const void *q, const void *k, const void *v, const int32_t *mask,
                             float scale, void *out, cudaStream_t st);
// bad_flag: device word that gets bit 0 set if a mask entry is >= the number of key blocks.
stream_status launch_vertical(const Geom &g, const int32_t *mask, const float *score, float *vertical, float *kurtosis,
                              unsigned int *bad_flag, cudaStream_t st);
stream_status launch_mask_diff(long long n_rows, int k_a, const int32_t *mask_a, const float *score_a, int k_b,
                               const int32_t *mask_b, int32_t *diff, float *diff_score, cudaStream_t st);
// Drains `st` and copies the tensor-core attention kernel's status words (code, block) to out.
stream_status read_attn_status(unsigned int out[2], cudaStream_t st);

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// Levels until every node is a single block: nodes start with at most ceil(N_k / k) blocks and
// the larger half of n blocks has ceil(n / 2). With N_k > 1 the first level always runs (it is
// where scores are first computed), matching n_it = ceil(log2 N_k) >= 1.
__host__ __device__ inline int levels_for(int N_k, int k) {
    long long sz = ((long long)N_k + k - 1) / k;
    int levels = 0;
    while (sz > 1) { sz = (sz + 1) / 2; ++levels; }
    return N_k > 1 ? (levels > 1 ? levels : 1) : 0;
}

// The sparsity constant of query block qb.
__device__ __forceinline__ int row_k(const Geom &g, int qb) {
    if (g.k_override > 0) return g.k_override;
    if (g.k_row == nullptr) return g.k_top;
    const int k = g.k_row[qb];
    return k < 1 ? 1 : (k > g.k_top ? g.k_top : k);
}

// Split levels of a row that runs with k = kq.
__host__ __device__ inline int row_levels(const Geom &g, int kq) {
    return kq == g.k_top ? g.levels : levels_for(g.N_k, kq);
}

// Last key block a row may look at (C^blk of Algorithm 2 in closed form), -1 if none.
__host__ __device__ inline int last_valid_block(const Geom &g, int qb) {
    long long last_tok = g.causal ? ((long long)qb * g.bq + g.bq - 1) : (g.T - 1);
    if (last_tok > g.T - 1) last_tok = g.T - 1;
    return (int)(last_tok / g.bk);
}

}  // namespace stream
