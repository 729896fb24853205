// Per-token Stream masks on the tensor cores for sm_100a: block_q = 1 (every query token is a row
// of its own), block_k = 64, bf16, d = 128, k_top <= 32 (Algorithm 2 at its finest query
// granularity, the [heads, T, k] shape of the mask).
//
// A row's candidate tile is now 1 x 64 x 128: eight thousand multiply-adds for 16 KB of keys,
// and every token has candidates of its own from the second level on. Gathering them token by
// token would move 128 times more key bytes than the contraction can use. Instead one CTA takes
// 128 consecutive tokens of one head through the hierarchy together, level by level:
//   - the tokens' candidate blocks of the level are merged into one ascending list (a bitmap over
//     the key blocks, set by the tokens, compacted by one warp);
//   - every block of the list is fetched once by TMA (two per stage) and multiplied with all 128
//     tokens at once: tcgen05.mma, A = the group's Q tile (128 tokens, shared memory), B = the pair
//     of key tiles (N = 128), fp32 accumulators in TMEM (128 columns per stage);
//   - a thread per token reads its lane of the accumulator, takes the masked maximum over each
//     tile's 64 keys (Eq. 4 under C, token level) and keeps it if that block is one of the
//     token's own candidates (a cursor over the token's ascending nodes);
//   - then each token ranks its 2k branch scores (higher score, then lower block index), keeps k,
//     and marks its next candidates in the bitmap.
// At the first level all tokens share the candidates; deeper down the merged list approaches
// "every block at the level's stride", so the work is that of a dense Q K^T restricted to the
// strides, at tensor-core rate, and each key tile crosses L2 -> SM once per 128 tokens.
//
// Roles (512 threads): warp 0 TMA producer and list builder, warps 1 and 3 issue the MMAs of the
// even and odd stages (warp 1 owns TMEM), warps 4..7 and 8..11 read the accumulators of the even
// and odd stages (thread = token). All sixteen warps take part in the per-token ranking, eight
// tokens each. The levels are separated by CTA-wide barriers; inside a level the roles meet on
// mbarriers, every wait bounded as in the other tensor-core kernels.
#include <math_constants.h>

#include "tc_common.cuh"

namespace stream {
namespace {

using namespace tc;

constexpr int kThreads = 512;
constexpr int kTok = 128;                    // tokens per group = rows of the A operand
constexpr int kBlk = 64, kD = 128;
constexpr int kStages = 4;                   // key-pair stages in shared memory = accumulator slots in TMEM
constexpr int kHalfTile = kBlk * 128;        // 64 keys x 128 bytes (one 64-channel half)
constexpr int kStageBytes = 4 * kHalfTile;   // [2 channel halves][2 tiles]
constexpr int kQBytes = 2 * kTok * 128;      // [2 channel halves][128 tokens][128 bytes]
constexpr int kPad = kTok + 1;               // row length of the per-token arrays (no bank conflicts either way)
constexpr int kMaxNk = 32768;                // key blocks (bitmap of 4 KB, block ids in 16 bits)
constexpr int kMaxList = kTok * 32;          // a level's merged list cannot be longer

struct Tail {
    unsigned long long full[kStages], empty[kStages], tmem_full[kStages], tmem_empty[kStages], q_full;
    unsigned int tmem_base;
    int abort_flag;
    int item;            // the group being worked on
    int n_list;          // blocks in the current level's list
    int n_nodes[kTok];   // surviving nodes per token
    int n_tiles[kTok];   // tiles the token has needed so far (its own candidates, not the merged list)
};

// Dynamic shared memory behind the 1024-byte aligned base:
//   Q tile | key-pair stages | scores [64][kPad] f32 | nodes [32][kPad] u32 | list u16 | bitmap u32 | Tail
// scores rows 0..31: score of a token's node j (its first allowed block); rows 32..63: score of
// node j's right branch at the current level. At the first level the 64 rows hold the scores of
// the (shared) list positions instead. nodes: first block | (blocks in the node << 16).
constexpr int kScoresBytes = 64 * kPad * 4, kNodesBytes = 32 * kPad * 4, kListBytes = kMaxList * 2, kBitmapBytes = kMaxNk / 8;
constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kScoresBytes + kNodesBytes + kListBytes + kBitmapBytes +
                           (int)sizeof(Tail) + 1024;
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");

constexpr unsigned kDescHi = desc_hi_sw128(1024);            // K-major, 8-row groups 1024 bytes apart
constexpr unsigned kIdesc = idesc_bf16(128, 128, false);     // D fp32, A and B bf16 K-major, M = N = 128

struct Params {
    Geom g;
    int n_items, n_tb;   // groups; groups per head (ceil(T / 128))
    int32_t *mask;
    float *score;
    WorkspaceHeader *ws;
};

__device__ __forceinline__ bool wait_w(unsigned bar, unsigned parity, Tail *tl, WorkspaceHeader *ws, unsigned code) {
    return mbar_wait_warp(bar, parity, &tl->abort_flag, &ws->error, &ws->error_info, code);
}

__device__ __forceinline__ unsigned pack_node(int f, int len) { return (unsigned)f | ((unsigned)len << 16); }

__global__ void __launch_bounds__(kThreads, 1)
mask_tok_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k, Params P) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const unsigned q_smem = smem_u32(smem), k_smem = q_smem + kQBytes;
    float *scores = (float *)(smem + kQBytes + kStages * kStageBytes);
    unsigned *nodes = (unsigned *)((unsigned char *)scores + kScoresBytes);
    unsigned short *list = (unsigned short *)((unsigned char *)nodes + kNodesBytes);
    unsigned *bitmap = (unsigned *)((unsigned char *)list + kListBytes);
    Tail *tl = (Tail *)((unsigned char *)bitmap + kBitmapBytes);
    const Geom &g = P.g;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const unsigned lt = (1u << lane) - 1u;

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(smem_u32(&tl->full[i]), 1); mbar_init(smem_u32(&tl->empty[i]), 1);
            mbar_init(smem_u32(&tl->tmem_full[i]), 1); mbar_init(smem_u32(&tl->tmem_empty[i]), 4);
        }
        mbar_init(smem_u32(&tl->q_full), 1);
        tl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    for (int i = tid; i < kMaxNk / 32; i += kThreads) bitmap[i] = 0u;
    if (warp == 1) tmem_alloc_512(smem_u32(&tl->tmem_base));  // all 512 columns (one CTA per SM)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = tl->tmem_base;

    // role of this warp inside a level
    const bool is_producer = warp == 0;
    const int mma_which = warp == 1 ? 0 : (warp == 3 ? 1 : -1);            // issues the stages with this parity
    const int epi_grp = (warp >= 4 && warp < 12) ? (warp - 4) >> 2 : -1;   // reads the stages with this parity
    const int epi_tok = (warp & 3) * 32 + lane;                            // its token (TMEM lane)

    const int kq = g.k_top, levels = g.levels;
    unsigned seq = 0;     // stages so far over the whole kernel (the same in every thread)
    unsigned q_par = 0;
    unsigned long long tiles_needed = 0, products = 0;  // per warp (lane 0 adds them up at the end)

    for (;;) {
        if (tid == 0) tl->item = (int)atomicAdd(&P.ws->work_counter, 1u);
        __syncthreads();
        const int id = tl->item;
        if (id >= P.n_items || *(volatile int *)&tl->abort_flag) break;
        // head by head (the keys of one kv head stay in L2), late token groups (most allowed blocks) first
        const int bh = id / P.n_tb, tb = P.n_tb - 1 - id % P.n_tb;
        const int b = bh / g.H, h = bh % g.H, kvh = h / g.hpg;
        const long long tok0 = (long long)tb * kTok;
        const long long tq_max = min(tok0 + kTok - 1, g.T - 1);
        const int q_lim_max = last_valid_block(g, (int)tq_max);

        if (is_producer) {
            if (elect_one()) {
                const unsigned bar = smem_u32(&tl->q_full);
                mbar_arrive_expect_tx(bar, (unsigned)kQBytes);
#pragma unroll
                for (int c = 0; c < 2; ++c) tma_load_4d(q_smem + c * (kQBytes / 2), &tmap_q, bar, c * 64, (int)tok0, h, b);
            }
            __syncwarp();
        }
        // initial nodes (the same for every token) and the first level's shared list
        const int f0 = (int)(((long long)lane * g.N_k) / kq), l0 = (int)(((long long)(lane + 1) * g.N_k) / kq) - 1;
        const int m0 = (f0 + l0) / 2;
        const bool gl = lane < kq && f0 <= l0 && f0 <= q_lim_max, gr = gl && m0 + 1 <= l0 && m0 + 1 <= q_lim_max;
        const unsigned bl = __ballot_sync(0xffffffffu, gl), br = __ballot_sync(0xffffffffu, gr);
        const int pos_l0 = __popc(bl & lt) + __popc(br & lt), pos_r0 = pos_l0 + (gl ? 1 : 0);
        if (warp == 0) {
            if (gl) list[pos_l0] = (unsigned short)f0;
            if (gr) list[pos_r0] = (unsigned short)(m0 + 1);
            if (lane == 0) tl->n_list = __popc(bl) + __popc(br);
        }
        // the token this thread reads accumulators for
        const long long e_tq = tok0 + epi_tok;
        const bool e_ok = epi_grp >= 0 && e_tq < g.T;
        const int e_qlim = e_ok ? last_valid_block(g, (int)e_tq) : -1;

        for (int level = 0; level < levels; ++level) {
            __syncthreads();  // the level's list is complete; the ranking of the level before is done
            const int n_list = tl->n_list, n_st = (n_list + 1) >> 1;

            if (is_producer) {
                for (int i = 0; i < n_st; ++i) {
                    const unsigned s = seq + (unsigned)i, buf = s & 3u;
                    if (!wait_w(smem_u32(&tl->empty[buf]), ((s >> 2) & 1u) ^ 1u, tl, P.ws, 601)) break;
                    const bool two = 2 * i + 1 < n_list;
                    const int blk0 = list[2 * i], blk1 = two ? list[2 * i + 1] : 0;
                    if (elect_one()) {
                        const unsigned bar = smem_u32(&tl->full[buf]), dst = k_smem + buf * kStageBytes;
                        mbar_arrive_expect_tx(bar, (unsigned)((two ? 4 : 2) * kHalfTile));
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            tma_load_4d(dst + c * 2 * kHalfTile, &tmap_k, bar, c * 64, blk0 * kBlk, kvh, b);
                            if (two) tma_load_4d(dst + (c * 2 + 1) * kHalfTile, &tmap_k, bar, c * 64, blk1 * kBlk, kvh, b);
                        }
                    }
                    __syncwarp();
                }
                if (lane == 0) products += 2ull * (unsigned long long)n_list;  // 128 tokens x 64 keys each
            } else if (mma_which >= 0) {
                bool ok = true;
                if (level == 0) ok = wait_w(smem_u32(&tl->q_full), q_par, tl, P.ws, 602);
                const unsigned a_lo = desc_lo_sw128(q_smem, 16);
                for (int i = 0; ok && i < n_st; ++i) {
                    const unsigned s = seq + (unsigned)i, buf = s & 3u, par = (s >> 2) & 1u;
                    if ((int)(s & 1u) != mma_which) continue;
                    if (!wait_w(smem_u32(&tl->full[buf]), par, tl, P.ws, 603)) break;
                    if (!wait_w(smem_u32(&tl->tmem_empty[buf]), par ^ 1u, tl, P.ws, 604)) break;
                    tc_fence_after();
                    const unsigned b_lo = desc_lo_sw128(k_smem + buf * kStageBytes, 16), d_tmem = tmem_base + buf * 128;
                    if (elect_one()) {
#pragma unroll
                        for (int c = 0; c < 2; ++c)
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4)
                                tc_mma_bf16_split(d_tmem, a_lo + ((c * (kQBytes / 2) + k4 * 32) >> 4), kDescHi,
                                                  b_lo + ((c * 2 * kHalfTile + k4 * 32) >> 4), kDescHi, kIdesc, (c | k4) != 0);
                        tc_commit(smem_u32(&tl->tmem_full[buf]));
                        tc_commit(smem_u32(&tl->empty[buf]));  // the stage is free once these MMAs have read it
                    }
                    __syncwarp();
                }
            } else if (epi_grp >= 0) {
                int cur = 0;  // cursor over this token's nodes (their right branches ascend with the list)
                const int n_nodes = level > 0 ? tl->n_nodes[epi_tok] : 0;
                for (int i = 0; i < n_st; ++i) {
                    const unsigned s = seq + (unsigned)i, buf = s & 3u;
                    if ((int)(s & 1u) != epi_grp) continue;
                    if (!wait_w(smem_u32(&tl->tmem_full[buf]), (s >> 2) & 1u, tl, P.ws, 605)) break;
                    tc_fence_after();
#pragma unroll
                    for (int tile = 0; tile < 2; ++tile) {
                        const int idx = 2 * i + tile;
                        if (idx >= n_list) break;  // (uniform)
                        const int blk = list[idx];
                        int pos = -1;  // where this token keeps the tile's score, if it is one of its candidates
                        if (level == 0) {
                            if (e_ok && blk <= e_qlim) pos = idx;
                        } else if (e_ok) {
                            while (cur < n_nodes) {
                                const unsigned nd = nodes[cur * kPad + epi_tok];
                                const int f = (int)(nd & 0xffffu), len = (int)(nd >> 16);
                                const int rb = (f + f + len - 1) / 2 + 1;
                                if (len > 1 && rb <= e_qlim) {
                                    if (rb == blk) pos = 32 + cur;
                                    if (rb >= blk) break;
                                }
                                ++cur;
                            }
                            if (pos >= 0) ++cur;
                        }
                        if (__any_sync(0xffffffffu, pos >= 0)) {
                            const unsigned taddr = tmem_base + buf * 128 + tile * 64 + ((unsigned)((warp & 3) * 32) << 16);
                            float v[64];
                            tmem_ld_32x32(taddr, v);
                            tmem_ld_32x32(taddr + 32, v + 32);
                            // keys of the block this token may look at: a prefix (inside T, not after the token if causal)
                            const long long k0 = (long long)blk * kBlk;
                            long long lim = g.T - k0;
                            if (g.causal) lim = min(lim, e_tq - k0 + 1);
                            const int n_hi = (int)max(0ll, min(lim, (long long)kBlk));
                            if (n_hi != kBlk) {  // the token's own block, or a block across T
#pragma unroll
                                for (int j = 0; j < 64; ++j) v[j] = j < n_hi ? v[j] : -CUDART_INF_F;
                            }
                            const float best = max_of_64(v);
                            if (pos >= 0) scores[pos * kPad + epi_tok] = best;
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&tl->tmem_empty[buf]));
                }
            }
            seq += (unsigned)n_st;
            if (level == 0) q_par ^= 1u;
            __syncthreads();  // every score of the level is in place
            if (*(volatile int *)&tl->abort_flag) break;  // (set only inside the level: the same answer in every thread)

            // ---- ranking: every warp takes eight tokens; lane j holds node j of the token ----
            const bool last = level + 1 == levels;
            for (int i = 0; i < kTok / (kThreads / 32); ++i) {
                const int t = warp * (kTok / (kThreads / 32)) + i;
                const long long tq = tok0 + t;
                if (tq >= g.T) break;  // (uniform) tokens beyond T: no row
                const int q_lim = last_valid_block(g, (int)tq);
                int f, l, m;
                bool vl, vr;
                float sl = -CUDART_INF_F, sr = -CUDART_INF_F;
                if (level == 0) {
                    f = f0; l = l0; m = m0;
                    vl = gl && f0 <= q_lim; vr = gr && m0 + 1 <= q_lim;
                    if (vl) sl = scores[pos_l0 * kPad + t];
                    if (vr) sr = scores[pos_r0 * kPad + t];
                    const int n0 = __popc(__ballot_sync(0xffffffffu, vl)) + __popc(__ballot_sync(0xffffffffu, vr));
                    if (lane == 0) { tiles_needed += (unsigned long long)n0; tl->n_tiles[t] = n0; }
                } else {
                    const int n = tl->n_nodes[t];
                    vl = lane < n;
                    const unsigned nd = vl ? nodes[lane * kPad + t] : pack_node(0, 0);
                    f = (int)(nd & 0xffffu); l = f + (int)(nd >> 16) - 1; m = (f + l) / 2;
                    vr = vl && l > f && m + 1 <= q_lim;
                    if (vl) sl = scores[lane * kPad + t];
                    if (vr) sr = scores[(32 + lane) * kPad + t];
                }
                const Keep kp = select_topk(vl, sl, vr, sr, kq, lane);
                const unsigned kl = __ballot_sync(0xffffffffu, kp.l), kr = __ballot_sync(0xffffffffu, kp.r);
                const int pos_l = __popc(kl & lt) + __popc(kr & lt), pos_r = pos_l + (kp.l ? 1 : 0);
                const int n_new = __popc(kl) + __popc(kr);
                __syncwarp();  // every lane has read its node and scores
                if (kp.l) { nodes[pos_l * kPad + t] = pack_node(f, m - f + 1); scores[pos_l * kPad + t] = sl; }
                if (kp.r) { nodes[pos_r * kPad + t] = pack_node(m + 1, l - m); scores[pos_r * kPad + t] = sr; }
                if (lane == 0) tl->n_nodes[t] = n_new;
                __syncwarp();
                const bool live = lane < n_new;
                const unsigned nn = live ? nodes[lane * kPad + t] : pack_node(0, 0);
                const int nf = (int)(nn & 0xffffu), nlen = (int)(nn >> 16);
                if (!last) {
                    // the token's candidates of the next level: the right branch of every node that has one
                    const int rb = (nf + nf + nlen - 1) / 2 + 1;
                    const bool has_r = live && nlen > 1 && rb <= q_lim;
                    if (has_r) atomicOr(&bitmap[rb >> 5], 1u << (rb & 31));
                    const unsigned hb = __ballot_sync(0xffffffffu, has_r);
                    if (lane == 0) { tiles_needed += (unsigned long long)__popc(hb); tl->n_tiles[t] += __popc(hb); }
                } else {
                    // emit I[token, :]: first block of every surviving node, ascending, -1 padded
                    const long long o = (((long long)b * g.H + h) * g.n_qb + tq) * g.k_top;
                    if (lane < g.k_top) {
                        P.mask[o + lane] = live ? nf : -1;
                        if (P.score != nullptr) P.score[o + lane] = live ? scores[lane * kPad + t] : -CUDART_INF_F;
                    }
                    if (g.row_tiles != nullptr && lane == 0)
                        g.row_tiles[((long long)b * g.H + h) * g.n_qb + tq] = (unsigned)tl->n_tiles[t];
                }
            }
            if (last) break;
            __syncthreads();  // the bitmap holds every token's candidates
            if (warp == 0) {  // compact it into the ascending list (and clear it for the level after)
                int base = 0;
                const int n_words = (g.N_k + 31) >> 5;
                for (int w0 = 0; w0 < n_words; w0 += 32) {
                    const int w = w0 + lane;
                    unsigned bits = w < n_words ? bitmap[w] : 0u;
                    if (w < n_words) bitmap[w] = 0u;
                    const int cnt = __popc(bits);
                    int incl = cnt;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int y = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += y;
                    }
                    int at = base + incl - cnt;
                    while (bits) {
                        const int bit = __ffs(bits) - 1;
                        bits &= bits - 1;
                        list[at++] = (unsigned short)(w * 32 + bit);
                    }
                    base += __shfl_sync(0xffffffffu, incl, 31);
                }
                if (lane == 0) tl->n_list = base;
            }
        }
        if (*(volatile int *)&tl->abort_flag) break;
        if (warp == 0 && lane == 0) atomicAdd(&P.ws->rows, (unsigned long long)(tq_max - tok0 + 1));
    }
    if (lane == 0 && (tiles_needed | products) != 0ull) {
        atomicAdd(&P.ws->tiles_scored, tiles_needed);
        atomicAdd(&P.ws->tile_products, products);
    }
    __syncwarp();

    // Teardown. After an abort, copies and MMAs may still be in flight: leave them a bounded time
    // to land before shared memory and TMEM are given back.
    if (*(volatile int *)&tl->abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_512(tmem_base);
    }
}

}  // namespace

bool mask_tok_supported(const Geom &g, int dtype) {
    return dtype == STREAM_BF16 && g.d == kD && g.bq == 1 && g.bk == kBlk && g.k_top <= 32 && g.levels >= 1 &&
           g.N_k <= kMaxNk && g.k_row == nullptr && g.k_override == 0 && tma_strides_ok(g);
}

stream_status launch_mask_tok(const Geom &g, const void *q, const void *k, int32_t *mask, float *score,
                              WorkspaceHeader *ws, cudaStream_t st) {
    if (((uintptr_t)q & 15) != 0 || ((uintptr_t)k & 15) != 0) {
        set_error("tensor-core mask kernel needs 16-byte aligned q and k");
        return STREAM_ERR_UNSUPPORTED;
    }
    CUtensorMap tq, tk;
    stream_status rc = make_map_bf16_d128(&tq, q, g.T, g.H, g.batch, g.qs_t, g.qs_h, g.qs_b, "q", kTok);
    if (rc != STREAM_OK) return rc;
    rc = make_map_bf16_d128(&tk, k, g.T, g.G, g.batch, g.ks_t, g.ks_h, g.ks_b, "k");
    if (rc != STREAM_OK) return rc;
    Params P;
    P.g = g;
    P.n_tb = (int)((g.T + kTok - 1) / kTok);
    const long long n_items = (long long)g.batch * g.H * P.n_tb;
    P.n_items = (int)n_items;
    P.mask = mask; P.score = score; P.ws = ws;
    const int n_sm = sm_count();
    if (n_sm <= 0) { set_error("cannot read the SM count of the current device"); return STREAM_ERR_CUDA; }
    cudaError_t e = cudaFuncSetAttribute(mask_tok_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(mask_tok)");
    const int grid = (int)(n_items < n_sm ? n_items : n_sm);
    mask_tok_kernel<<<grid, kThreads, kSmemBytes, st>>>(tq, tk, P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "mask_tok launch");
    return STREAM_OK;
}

}  // namespace stream
