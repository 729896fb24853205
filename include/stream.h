/*
 * libstream: C ABI of the B200 (sm_100a) implementation of Stream sparse-mask estimation and
 * the block-sparse attention pass that consumes the mask.
 *
 * Conventions for every entry point
 *   - Plain C types only. Unless a parameter says HOST, every data pointer is a DEVICE pointer
 *     owned by the caller; the library never allocates or frees device memory. The state it
 *     keeps between calls is: the thread-local error text; per device, the two copy streams and
 *     the events of stream_run_host (created at its first call, kept until the process ends);
 *     per device, the built-in scratch array of stream_build_mask_static and its address; and
 *     the status word of the tensor-core attention kernel (stream_check_device_status).
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and the call returns after enqueue unless stated otherwise.
 *   - Every failure is a returned status; nothing aborts or throws. Arguments are validated on
 *     the host before anything is launched. stream_last_error() gives the text of the last
 *     failure on the calling thread.
 *   - Tensors: Q is [batch, n_q_heads, T, d], K and V are [batch, n_kv_heads, T, d], addressed
 *     with the element strides in the problem struct (innermost stride 1). Query head h reads
 *     kv head h / (n_q_heads / n_kv_heads). dtype is fp32 or bf16 for Q, K, V and the attention
 *     output alike. Inputs must be finite.
 *   - A "row" is one (batch, query head, query block); there are ceil(T / block_q) query
 *     blocks. The mask is int32 [batch, n_q_heads, ceil(T / block_q), k_top], contiguous: per
 *     row the kept key-block indices (0-based; block r covers tokens r*block_k ..), strictly
 *     ascending, then -1 padding.
 */
#ifndef STREAM_H_
#define STREAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    STREAM_OK = 0,
    STREAM_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bad stride, bad enum */
    STREAM_ERR_UNSUPPORTED = 2, /* valid request that no kernel here covers (see stream_problem) */
    STREAM_ERR_WORKSPACE = 3,   /* workspace or staging buffer missing, misaligned or too small */
    STREAM_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; text in stream_last_error */
    STREAM_ERR_DEVICE_CHECK = 5 /* a kernel gave up on a bounded wait or met an out-of-range mask
                                   entry; see stream_read_stats */
} stream_status;

typedef enum { STREAM_F32 = 0, STREAM_BF16 = 1 } stream_dtype;

typedef enum {
    STREAM_IMPL_AUTO = 0,    /* tensor-core kernels when the shape allows, else the generic ones */
    STREAM_IMPL_GENERIC = 1, /* fp32-FMA kernels: any dtype, d in {16,32,64,128,256}, blocks 1..64 */
    STREAM_IMPL_TENSOR = 2   /* tcgen05 kernels only: bf16, d = 128, block_q = block_k = 64, strides
                                that are multiples of 8 elements, 16-byte aligned pointers (and
                                k_top <= 32 for the mask build); the mask build also takes
                                block_q = 1 (per-token masks) with block_k = 64, one k, and at most
                                32768 key blocks; otherwise STREAM_ERR_UNSUPPORTED */
} stream_impl;

typedef struct {
    int32_t batch;          /* independent problems (e.g. layers); >= 1 */
    int32_t n_q_heads;      /* >= 1 */
    int32_t n_kv_heads;     /* >= 1 and divides n_q_heads */
    int64_t T;              /* tokens, >= 1; need not be a multiple of the block sizes */
    int32_t d;              /* head dimension: 16, 32, 64, 128 or 256 */
    int32_t block_q;        /* b_q */
    int32_t block_k;        /* b_k */
    int32_t k_top;          /* k: key blocks kept per query block = row width of the mask; 1..1024 */
    int32_t causal;         /* 1: C is lower triangular; 0: C is all ones (Algorithm 1) */
    int32_t dtype;          /* stream_dtype */
    int32_t impl;           /* stream_impl */
    int64_t q_stride_b, q_stride_h, q_stride_t;    /* elements */
    int64_t kv_stride_b, kv_stride_h, kv_stride_t; /* elements; K and V share them */
} stream_problem;

/* Counters a mask build leaves in the first bytes of its workspace. */
typedef struct {
    uint64_t tiles_scored; /* (row, representative key block) tiles whose score was computed */
    uint64_t rows;         /* rows finished */
    uint32_t error;        /* 0, or a code saying which bounded wait ran out (kernel returned early) */
    uint32_t error_info;
    uint64_t tile_products; /* 64 x 64 x d tile products the per-token tensor-core kernel computed (it
                               multiplies every fetched key tile with 128 tokens at once, so this
                               exceeds tiles_scored / 64); 0 from the other kernels, whose products
                               are exactly the tiles scored */
    uint64_t tiles_fetched; /* key and query tiles (block x d) the tensor-core block kernel copied into
                               shared memory: fewer than tiles_scored where a fetched key tile serves
                               several rows; 0 from the kernels that do not count them */
} stream_stats;

/* Library version: major * 10000 + minor * 100 + patch. */
int stream_version(void);

/* Text of the most recent failure on this thread ("" if none). The pointer stays valid until the
 * thread's next failing call. */
const char *stream_last_error(void);

/*
 * Bytes of device workspace stream_build_mask needs for this problem (a small header holding
 * stream_stats and the work counter of the persistent kernels; O(1), never grows with T).
 * Returns 0 if the problem is invalid or unsupported.
 */
size_t stream_workspace_bytes(const stream_problem *p);

/*
 * Stream mask estimation (Algorithm 2 of the paper; Algorithm 1 when causal == 0).
 *
 * For every row: start from k_top nodes tiling the N_k key blocks, and for ceil(log2 N_k) levels
 * split every node in two, score each branch by the masked maximum token-level dot product
 * (Eq. 4) between the query block and the branch's first allowed key block, keep the k_top best
 * branches (higher fp32 score, then lower block index), and finally emit the first allowed block
 * of every surviving node. Levels that cannot change the result (all nodes single blocks) are
 * skipped, and a left branch reuses its parent's score (same tile, same value).
 *
 *   q, k       device, dtype of the problem, strided as described above; read only
 *   mask_out   device int32 [batch, n_q_heads, ceil(T/block_q), k_top]; fully overwritten
 *   score_out  device float32, same shape, or NULL: block score of every kept block, -inf padded
 *   workspace  device, 256-byte aligned, >= stream_workspace_bytes(p); overwritten. After the
 *              stream has drained, stream_read_stats(workspace, ...) returns this call's counters.
 *              If workspace_bytes >= stream_workspace_bytes(p) + 4 * rows (rows = batch *
 *              n_q_heads * ceil(T/block_q)), the build also writes, as uint32 [rows] right behind
 *              the first stream_workspace_bytes(p) bytes, how many tiles each row scored (their
 *              sum is stream_stats.tiles_scored). stream_build_mask and stream_build_mask_var only.
 *
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE before any launch; CUDA if a launch fails.
 */
stream_status stream_build_mask(const stream_problem *p, const void *q, const void *k, int32_t *mask_out,
                                float *score_out, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * stream_build_mask with a sparsity constant of its own for every query block ("variable k": the
 * paper's discussion of needle depth, Section 4.2, and the fourth item of its Limitations name it
 * as the remedy for the stronger pruning of late rows under a causal mask, and leave it
 * undefined). The reading taken: the row of query block qb is Algorithm 2, unchanged, run with
 * k = k_row[qb]; rows stay k_top wide (the row's blocks ascending, then -1; scores -inf padded),
 * so the result feeds stream_sparse_attention, stream_vertical_scores and stream_mask_difference
 * as it is.
 *
 *   k_row      device int32 [ceil(T/block_q)], shared by all heads and batch entries; read only.
 *              Entries outside 1 .. k_top are clamped into that range.
 * Everything else as stream_build_mask (p->k_top is the row width and the largest k).
 */
stream_status stream_build_mask_var(const stream_problem *p, const void *q, const void *k, const int32_t *k_row,
                                    int32_t *mask_out, float *score_out, void *workspace, size_t workspace_bytes,
                                    void *cuda_stream);

/*
 * The masks of the same inputs for several sparsity constants in one call: the search over k of
 * Section 3 (binary search for the smallest k that keeps the model's behaviour) and the
 * k_success / k_fail comparison of Section 4.2 need them. Mask i is Algorithm 2 with
 * k = k_list_host[i]. A block's score does not depend on k, so where the kernel can keep a row's
 * scores (the generic kernel, while ceil(T/block_k) floats fit in shared memory beside its tiles)
 * every (row, block) tile is scored once for all k. The tensor-core kernel does the same when the
 * workspace has room for its score memory (stream_workspace_bytes_multi: 8 bytes per key block, row
 * of a group and SM, i.e. O(T)); with only stream_workspace_bytes it is launched once per k and
 * shares nothing. stream_read_stats then reports the tiles actually scored over the whole call.
 *
 *   n_k          1 .. 8
 *   k_list_host  HOST int32 [n_k], each 1 .. p->k_top (p->k_top is the row width), any order
 *   mask_out     device int32 [n_k, batch, n_q_heads, ceil(T/block_q), k_top]; mask i is one
 *                contiguous slab, its rows -1 padded beyond k_list_host[i] entries
 *   score_out    device float32, same shape, or NULL
 * Everything else, and the errors, as stream_build_mask.
 */
size_t stream_workspace_bytes_multi(const stream_problem *p, int32_t n_k);  /* 0 = invalid problem or n_k */
stream_status stream_build_mask_multi(const stream_problem *p, const void *q, const void *k, int32_t n_k,
                                      const int32_t *k_list_host, int32_t *mask_out, float *score_out, void *workspace,
                                      size_t workspace_bytes, void *cuda_stream);

/*
 * A schedule for stream_build_mask_var, computed on the host: the effective-sparsity formula of
 * Section 4.2, k = floor(1 + (n - 1) s), applied per query block with n = the number of key
 * blocks that row may look at (qb + 1 blocks under a causal mask with equal block sizes; the
 * paper applies the formula once, with n = T / b_q, which is what prunes late rows harder).
 * Clamped to 1 .. p->k_top.
 *
 *   s           0 < s < 1, else INVALID_ARG
 *   k_row_host  HOST int32 [ceil(T/block_q)], overwritten; copy it to the device for the build
 */
stream_status stream_k_schedule(const stream_problem *p, double s, int32_t *k_row_host);

/*
 * The effective-sparsity formula of Section 4.2 as printed: k = floor(1 + (T / b_q - 1) s), kept
 * inside k's range 1 .. floor(T / b_q) (at least 1). T / b_q is taken as the real quotient. As
 * printed, a larger s keeps MORE blocks (the prose beside the formula says the opposite; the
 * formula is followed). Host-only arithmetic; nothing is launched.
 *
 *   s           0 <= s <= 1, else INVALID_ARG
 *   k_out_host  HOST int32, one value
 */
stream_status stream_effective_k(int64_t T, int32_t block_q, double s, int32_t *k_out_host);

/*
 * stream_build_mask without a caller-provided workspace and without any allocation. (The paper
 * has no counterpart to this entry point; it exists for deployment.)
 *
 * For callers that cannot get device memory when they call: a host application that reserved all
 * of HBM for its own pool at start-up, or a latency-critical loop that must not hit the implicit
 * synchronisation of cudaMalloc / cudaFree. The kernel's scratch (work counter and counters, see
 * stream_stats) lives in a 4096-byte device array built into the library, which each GPU that
 * loads the library holds until the process exits. Same arguments, results and errors as
 * stream_build_mask otherwise (an invalid or unsupported problem gets exactly the status
 * stream_build_mask gives it); a problem whose scratch need exceeded 4096 bytes would be refused
 * with STREAM_ERR_WORKSPACE (no current problem does). The call allocates and frees nothing.
 *
 *   - The first call on each device looks up the array's device address (a one-time host-side
 *     query, made with that device current). Make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents; each
 *     call clears what it needs on `cuda_stream` before its kernel. Two calls that can overlap on
 *     the GPU (different streams, no dependency) race on it: serialise them, or give the
 *     overlapping calls stream_build_mask with workspaces of their own.
 *   - The counters are not readable through this entry point.
 */
stream_status stream_build_mask_static(const stream_problem *p, const void *q, const void *k, int32_t *mask_out,
                                       float *score_out, void *cuda_stream);

/*
 * Block-sparse attention under a Stream mask (Eq. 2 of the paper; the product QK^T * C * M of
 * Figure 1): for every query token, softmax(scale * q.k) over the keys of the row's kept blocks
 * that C allows (element-level causal test inside a block, keys beyond T excluded), times V.
 * Softmax statistics and the output accumulate in fp32; a token that no kept key is allowed for
 * gets zeros.
 *
 *   q, k, v    device, dtype of the problem; read only
 *   mask       device int32 [batch, n_q_heads, ceil(T/block_q), k_top] as written by
 *              stream_build_mask; entries < 0 are skipped; valid entries must be < ceil(T/block_k)
 *   scale      logit scale; <= 0 selects 1/sqrt(d)
 *   out        device, dtype of the problem, contiguous [batch, n_q_heads, T, d]; overwritten
 */
stream_status stream_sparse_attention(const stream_problem *p, const void *q, const void *k, const void *v,
                                      const int32_t *mask, float scale, void *out, void *cuda_stream);

/*
 * Vertical attention scores of a mask and their kurtosis (Section 4.1 of the paper: the column
 * sums of a head's sparse mask show which key blocks attract the later queries; heads whose
 * vertical scores have a high kurtosis are the "receiver heads").
 *
 *   vertical[b, h, r] = sum over the head's query blocks q and slots j with mask[b, h, q, j] == r
 *                       of scores[b, h, q, j]   (of 1 if scores is NULL: the binary mask)
 *   kurtosis[b, h]    = m4 / m2^2 of vertical[b, h, :], m2 and m4 the second and fourth central
 *                       moments over the ceil(T / block_k) key blocks (Pearson, not excess); 0
 *                       if all vertical scores of the head are equal
 *
 *   mask          device int32 [batch, n_q_heads, ceil(T/block_q), k_top]; entries < 0 are skipped
 *   scores        device float32, same shape (score_out of stream_build_mask), or NULL; -inf
 *                 padding is never read because its mask entry is < 0
 *   vertical_out  device float32 [batch, n_q_heads, ceil(T/block_k)]; overwritten
 *   kurtosis_out  device float32 [batch, n_q_heads], or NULL
 *   workspace     as for stream_build_mask; stream_read_stats afterwards returns
 *                 STREAM_ERR_DEVICE_CHECK if a mask entry was >= ceil(T/block_k) (such entries
 *                 are ignored). Sums are fp32 and added in no fixed order.
 * Only T, block_k, block_q, k_top, batch and n_q_heads of *p matter. Up to 49152 key blocks per
 * head; more gives STREAM_ERR_UNSUPPORTED.
 */
stream_status stream_vertical_scores(const stream_problem *p, const int32_t *mask, const float *scores, float *vertical_out,
                                     float *kurtosis_out, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Mask subtraction (Section 4.2 of the paper, "Exploring Information Flow": the sparse masks
 * found with a smaller budget k are subtracted from those found with a larger one; what is left,
 * weighted by the larger mask's block scores, are the connections only the larger budget keeps).
 * Row by row: the entries of mask_a that are >= 0 and do not occur in the same row of mask_b, in
 * mask_a's order, then -1 padding (their scores, then -inf padding).
 *
 *   n_rows           rows of both masks (batch * n_q_heads * query blocks)
 *   mask_a, mask_b   device int32 [n_rows, k_a] and [n_rows, k_b], 1 <= k_a, k_b <= 1024; any order
 *   scores_a         device float32 [n_rows, k_a] or NULL
 *   diff_out         device int32 [n_rows, k_a]; overwritten; must not alias the inputs
 *   diff_scores_out  device float32 [n_rows, k_a] or NULL (needs scores_a)
 */
stream_status stream_mask_difference(int64_t n_rows, int32_t k_a, const int32_t *mask_a, const float *scores_a, int32_t k_b,
                                     const int32_t *mask_b, int32_t *diff_out, float *diff_scores_out, void *cuda_stream);

/*
 * Synchronous read-back of the counters left by the last stream_build_mask that used this
 * workspace. Waits for `cuda_stream` to drain, copies the header to *out (HOST pointer) and
 * returns STREAM_ERR_DEVICE_CHECK if the kernel recorded a failed device-side check (a bounded
 * wait that ran out; an out-of-range mask entry in stream_vertical_scores).
 */
stream_status stream_read_stats(const void *workspace, stream_stats *out, void *cuda_stream);

/*
 * Synchronous health check of the kernels that have no workspace to report into (the tensor-core
 * attention kernel). Waits for `cuda_stream` to drain and returns STREAM_ERR_DEVICE_CHECK if, on
 * the current device and since the library was loaded, such a kernel gave up on one of its
 * bounded waits and left early (its output is then incomplete); STREAM_OK otherwise.
 */
stream_status stream_check_device_status(void *cuda_stream);

/*
 * Diagnostic (the paper has no counterpart): runs the bounded wait that every mbarrier wait of the
 * tensor-core kernels goes through to its limit once, in a one-warp kernel of its own that waits
 * on a barrier nothing arrives at, with no copy or tensor-core operation in flight. After
 * limit_cycles SM clock cycles the wait gives up exactly as it would in a product kernel: it
 * records code 901 in the workspace header, raises the abort flag, all lanes leave together and
 * the kernel returns. stream_read_stats(workspace, ...) then returns STREAM_ERR_DEVICE_CHECK with
 * error = 901 (rows = 0: the wait did not succeed; tiles_scored = 1: the abort flag was raised).
 * The product kernels use the same code path with a limit of 2^31 cycles (about a second).
 *
 *   limit_cycles  1 .. 2^31, else INVALID_ARG
 *   workspace     device, 256-byte aligned, >= 256 bytes; overwritten
 */
stream_status stream_selftest_bounded_wait(int64_t limit_cycles, void *workspace, size_t workspace_bytes,
                                           void *cuda_stream);

/* What stream_probe_unit_rates measured. */
typedef struct {
    double tma_bytes_per_clk;   /* bytes per SM clock that one SM's TMA unit brought from L2 into its shared
                                   memory (16 KiB bulk copies of L2-resident data, two issuing warps with
                                   four copies in flight each, every SM busy at once; CTA 0's figure) */
    double mma_cycles_m128n64;  /* SM clocks per tcgen05.mma of M = 128, N = 64, K = 16, bf16, shared-memory
                                   operands, issued back to back (32 would be the tensor core's own time) */
    uint32_t error;             /* 0, or the code of a bounded wait that ran out (911 copies, 912 MMAs) */
    uint32_t reserved;
} stream_unit_rates;

/*
 * Measurement aid (the paper has no counterpart): the two unit rates that bound the tensor-core
 * mask and attention kernels on the device at hand, so that a measured throughput can be set
 * against what the SM delivers rather than against a data-sheet figure. Launches two short
 * kernels (one CTA per SM, a few hundred microseconds), waits for `cuda_stream` and fills
 * *out_host. Every wait inside is bounded like the product kernels' (STREAM_ERR_DEVICE_CHECK and
 * out_host->error if one ran out).
 *
 *   scratch       device, 256-byte aligned, >= stream_probe_scratch_bytes(); overwritten (zeros:
 *                 the source of the copies and a result record)
 *   out_host      host
 */
size_t stream_probe_scratch_bytes(void);
stream_status stream_probe_unit_rates(void *scratch, size_t scratch_bytes, stream_unit_rates *out_host, void *cuda_stream);

/*
 * Bytes of device staging stream_run_host and stream_run_host_var need: room for Q, K, V, the mask,
 * the output, the mask workspace and one k per query block, each 256-byte aligned. 0 if the problem
 * is invalid or unsupported.
 */
size_t stream_host_staging_bytes(const stream_problem *p);

/*
 * The whole path from HOST memory: copy Q, K, V to the device, build the mask, run the sparse
 * attention, copy mask and output back. Strides in *p describe the HOST tensors, which must be
 * dense ([batch, heads, T, d] contiguous). The work is cut into one chunk per (batch entry, kv
 * head) - nothing else depends on a chunk - and chunk c + 1's copy in, chunk c's kernels and
 * chunk c - 1's copy out run at the same time: the copies on two streams the library creates
 * once per device at the first call (with a few events; kept until the process ends), the
 * kernels on cuda_stream. Pinned host memory is what makes the copies asynchronous.
 *
 *   q_host, k_host, v_host   HOST, read only
 *   mask_host                HOST int32 [batch, n_q_heads, ceil(T/block_q), k_top]
 *   out_host                 HOST, dtype of the problem, [batch, n_q_heads, T, d]
 *   staging                  DEVICE, 256-byte aligned, >= stream_host_staging_bytes(p)
 * Everything is ordered after what cuda_stream already holds, and cuda_stream is made to wait
 * for the last copy out: the host buffers are valid once cuda_stream has been synchronised. Two
 * calls that share a device must not overlap in time (they share the internal streams' events).
 */
stream_status stream_run_host(const stream_problem *p, const void *q_host, const void *k_host, const void *v_host,
                              int32_t *mask_host, void *out_host, float scale, void *staging,
                              size_t staging_bytes, void *cuda_stream);

/*
 * stream_run_host with a sparsity constant of its own for every query block (the variable-k build
 * of stream_build_mask_var, Section 4.2's remedy for the harder pruning of late rows, followed by
 * the sparse attention on its masks), from HOST memory and pipelined the same way.
 *
 *   k_row_host   HOST int32 [ceil(T/block_q)], e.g. from stream_k_schedule; entries outside
 *                1 .. k_top are clamped. It is copied to the staging buffer ahead of the first chunk.
 * Everything else as stream_run_host (same staging size).
 */
stream_status stream_run_host_var(const stream_problem *p, const void *q_host, const void *k_host, const void *v_host,
                                  const int32_t *k_row_host, int32_t *mask_host, void *out_host, float scale, void *staging,
                                  size_t staging_bytes, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* STREAM_H_ */
