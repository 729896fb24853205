// Tensor-core block-sparse attention for sm_100a (Eq. 2 on a Stream mask): bf16, d = 128,
// 64 x 64 blocks.
//
// One persistent CTA per SM works through "pairs": two query heads of one kv head at one query
// block. Their Q tiles are stacked into one 128-row A operand. For every mask entry e the two
// rows name one key block each (K_a, K_b, usually different); the tiles arrive by TMA (128-byte
// swizzle), stacked too, and
//     S = [Q_0; Q_1] [K_a; K_b]^T      (128 x 128, fp32 in TMEM)
// holds row 0's logits in its upper-left quadrant and row 1's in its lower-right one. The
// softmax warps own one TMEM lane (= one query token) per thread pair: they read its 64 logits,
// apply the element-level mask C, update the running maximum and sum (online softmax, fp32), and
// write P = exp(.) as bf16 into a block-diagonal 128 x 128 A operand in shared memory whose
// off-diagonal quadrants stay zero. Then
//     O_e = P [V_a; V_b]               (128 x 128, fp32 in TMEM, V tiles MN-major)
// gives both rows' contributions in one chain, which the same threads fold into their fp32
// output registers (o = o * alpha + O_e) one iteration later, so that the tensor core works on
// the next logits meanwhile.
//
// Roles (384 threads): warp 0 TMA producer (converged, one elected lane issues); warp 1 issues the Q K^T chains and owns TMEM; warp 3
// issues the P V chains (two issuing warps, because the thread that issues a chain is held until
// the tensor core has taken it: with one warp the waits and commits between chains would not
// overlap with the chains themselves); warp 2 copies the pairs' mask rows from global to shared
// memory ahead of everyone else; warps 4..11 softmax (two threads per query token: half of its
// keys and half of its output channels each). Every role walks the same sequence of (pair,
// entry), read from the shared copy of the mask rows; they meet only on mbarriers. Every wait is
// bounded: on a timeout the CTA records a code in a device status word, raises a shared abort
// flag, lets its copies drain and leaves.
#include <math_constants.h>

#include "tc_common.cuh"

namespace stream {

// Status word of the tensor-core attention kernel: 0, or the code of the bounded wait that ran
// out (with the block index beside it). Read by stream_check_device_status.
__device__ unsigned int g_attn_status[2];

namespace {

using namespace tc;

constexpr int kThreads = 384;
constexpr int kBlk = 64, kD = 128;
constexpr int kHalfTile = kBlk * 128;       // 64 rows x 128 bytes
constexpr int kTile = 2 * kHalfTile;        // one 64 x 128 tile
constexpr int kOperand = 2 * kTile;         // two tiles (K_a, K_b or V_a, V_b), or a 128-row operand
constexpr int kMaxKStages = 3, kVStages = 2;  // K stages: 3 if shared memory allows, else 2; V stages = O buffers
constexpr int kMaskSlots = 2;               // pairs whose mask rows are resident
constexpr int kMaxKTopTc = 1024;

struct Tail {
    unsigned long long q_full, q_empty;
    unsigned long long k_full[kMaxKStages], k_empty[kMaxKStages], v_full[kVStages];
    // o_full also tells the producer that V stage i is free: the rings of V stages and O buffers
    // have the same length and move together. There is no "o_empty": P of entry j is published
    // (p_full) after the same threads folded the product of entry j - 2, and the P V warp waits
    // for every P before it overwrites that buffer.
    unsigned long long s_full[2], s_empty[2], o_full[2], p_full;
    unsigned long long m_full[kMaskSlots], m_empty[kMaskSlots];
    unsigned long long x_bar[4];  // softmax warps w and w + 4 meet here
    unsigned int tmem_base;
    int abort_flag;
    float xch[2][128][2];         // their exchange slots: [buffer][token][part]
};
// Dynamic shared memory: Q | P | V stages | K stages | Tail | mask rows [kMaskSlots][2][row_stride]
// (-1 where a row has nothing), the first four 1024-byte aligned.
constexpr int kFixedOperands = 2 + kVStages;
constexpr int kMaxSmemPerCta = 232448;

constexpr unsigned kIdescQK = idesc_bf16(128, 128, false);  // B = stacked K tiles, K-major
constexpr unsigned kIdescPV = idesc_bf16(128, 128, true);   // B = stacked V tiles, MN-major
constexpr unsigned kHiK = desc_hi_sw128(1024);              // every operand: 8-row (8-key) groups 1024 bytes apart

struct Params {
    Geom g;
    int n_items, n_pairs;  // pairs per kv head: ceil(hpg / 2)
    int row_stride;        // ints per resident mask row (k_top rounded up to a multiple of 4)
    int smem_bytes;        // dynamic shared memory of the launch
    int n_k_stages;        // set by the kernel from what fits behind its aligned base
    const int32_t *mask;
    __nv_bfloat16 *out;
    float scale_log2;      // logit scale times log2(e)
};

__device__ __forceinline__ bool wait(unsigned bar, unsigned parity, Tail *tl, unsigned code) {
    return mbar_wait_bounded(bar, parity, &tl->abort_flag, &g_attn_status[0], &g_attn_status[1], code);
}

// The same for a whole converged warp (all lanes get the same answer).
__device__ __forceinline__ bool wait_w(unsigned bar, unsigned parity, Tail *tl, unsigned code) {
    return mbar_wait_warp(bar, parity, &tl->abort_flag, &g_attn_status[0], &g_attn_status[1], code);
}

// Shared copy of the mask rows of the pair in slot `slot`: [2][row_stride] ints behind the Tail.
__device__ __forceinline__ int *mask_rows(Tail *tl, const Params &P, int slot) {
    return reinterpret_cast<int *>(tl + 1) + slot * 2 * P.row_stride;
}

// The pair a CTA works on in its n-th round.
struct Item {
    int b, kvh, qb, h0, R;
};

__device__ __forceinline__ Item decode_item(const Params &P, int id) {
    const Geom &g = P.g;
    Item it;
    // kv head by kv head, so that the K and V tiles in flight belong to one head at a time (64 MiB
    // at T = 131072: they stay in L2); within a head late query blocks (most kept blocks under a
    // causal mask) first
    const int per_head = g.n_qb * P.n_pairs;
    const int bh = id / per_head;
    const int rem = id % per_head;
    it.qb = g.n_qb - 1 - rem / P.n_pairs;
    const int pair = rem % P.n_pairs;
    it.kvh = bh % g.G;
    it.b = bh / g.G;
    it.h0 = it.kvh * g.hpg + pair * 2;
    it.R = min(2, g.hpg - pair * 2);
    return it;
}

// Entry e of the two rows: key block per row (negative = this row has nothing at e). An entry
// is processed if either row has a block there. `rows` is the pair's shared copy [2][stride].
struct Entry { int a, b; };
__device__ __forceinline__ int next_entry(const int *rows, int stride, int e, int k_top, Entry *x) {
    for (++e; e < k_top; ++e) {
        x->a = rows[e];
        x->b = rows[stride + e];
        if (x->a >= 0 || x->b >= 0) return e;
    }
    return k_top;
}

// ----------------------------------------------------------------------------------------------
// Roles. All walk the kept entries x_0 .. x_{n-1} of a pair in "rounds": round r handles the
// logits of x_r and the P V product of x_{r-1}.
// ----------------------------------------------------------------------------------------------
__device__ void mask_loader_role(const Params &P, Tail *tl, int lane) {
    const Geom &g = P.g;
    Ring ms;
    for (int id = blockIdx.x; id < P.n_items; id += gridDim.x) {
        const Item it = decode_item(P, id);
        if (!wait(smem_u32(&tl->m_empty[ms.idx]), ms.phase ^ 1, tl, 401)) return;
        const int32_t *m0 = P.mask + (((long long)it.b * g.H + it.h0) * g.n_qb + it.qb) * g.k_top;
        const int32_t *m1 = m0 + (long long)g.n_qb * g.k_top;
        int *dst = mask_rows(tl, P, ms.idx);
        for (int e = lane; e < g.k_top; e += 32) {
            dst[e] = __ldg(m0 + e);
            dst[P.row_stride + e] = it.R == 2 ? __ldg(m1 + e) : -1;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&tl->m_full[ms.idx]));
        ms.advance(kMaskSlots);
    }
}

// One warp feeds two independent streams of TMA loads, the K tiles (with each pair's Q tiles)
// and the V tiles, each as far ahead as its ring of stages allows. It never blocks on one stream
// while the other could move: every step probes its barrier without waiting. The warp runs
// converged (lane 0's probe result is broadcast) and one elected lane issues.
struct LoadStream {
    int id;            // pair being walked
    int e;             // current entry (k_top = pair exhausted), -2 = pair not opened yet
    int n_issued;      // loads issued for this pair
    Entry cur;
    Item it;
    Ring ring, ms;
    bool q_due;        // (K stream) the pair's Q tiles still have to be requested
};

__device__ __forceinline__ bool probe_w(unsigned bar, unsigned parity) {
    return __shfl_sync(0xffffffffu, (int)mbar_test_wait(bar, parity), 0) != 0;
}

__device__ void producer_role(const Params &P, const CUtensorMap *tq, const CUtensorMap *tk, const CUtensorMap *tv,
                              Tail *tl, unsigned q_smem, unsigned k_smem, unsigned v_smem) {
    const Geom &g = P.g;
    unsigned q_par = 0;
    LoadStream K, V;
    K.id = V.id = blockIdx.x;
    K.e = V.e = -2;
    K.q_due = V.q_due = false;
    // a row without a block at an entry gets block 0; its logits are masked out entirely
    auto load_k_pair = [&](unsigned dst, unsigned bar, const Item &it, Entry x) {  // [half][tile][64 rows][128 B]
        const int ba = x.a >= 0 ? x.a : 0, bb = x.b >= 0 ? x.b : 0;
        mbar_arrive_expect_tx(bar, (unsigned)kOperand);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            tma_load_4d(dst + c * 2 * kHalfTile, tk, bar, c * 64, ba * kBlk, it.kvh, it.b);
            tma_load_4d(dst + c * 2 * kHalfTile + kHalfTile, tk, bar, c * 64, bb * kBlk, it.kvh, it.b);
        }
    };
    auto load_v_pair = [&](unsigned dst, unsigned bar, const Item &it, Entry x) {  // [tile][half][64 rows][128 B]
        const int ba = x.a >= 0 ? x.a : 0, bb = x.b >= 0 ? x.b : 0;
        mbar_arrive_expect_tx(bar, (unsigned)kOperand);
        tma_load_5d(dst, tv, bar, 0, ba * kBlk, it.kvh, 0, it.b);
        tma_load_5d(dst + kTile, tv, bar, 0, bb * kBlk, it.kvh, 0, it.b);
    };
    // One step of a stream; true if it did something. is_k selects the K (+ Q) or the V stream.
    auto step = [&](LoadStream &S, bool is_k) -> bool {
        if (S.id >= P.n_items) return false;
        const int *rows = mask_rows(tl, P, S.ms.idx);
        if (S.e == -2) {  // open the pair: its mask rows must be resident
            if (!probe_w(smem_u32(&tl->m_full[S.ms.idx]), S.ms.phase)) return false;
            S.it = decode_item(P, S.id);
            S.e = next_entry(rows, P.row_stride, -1, g.k_top, &S.cur);
            S.q_due = is_k && S.e < g.k_top;  // (a pair with nothing kept: only the softmax warps act)
            S.n_issued = 0;
            return true;
        }
        if (S.e >= g.k_top && !S.q_due) {  // pair exhausted: give its mask rows back, go to the next one
            if (elect_one()) mbar_arrive(smem_u32(&tl->m_empty[S.ms.idx]));
            __syncwarp();
            S.ms.advance(kMaskSlots);
            S.id += gridDim.x;
            S.e = -2;
            return true;
        }
        if (is_k) {
            if (S.e < g.k_top && !(S.q_due && S.n_issued > 0)) {
                // a K stage is free once the logits computed from it are complete
                if (!probe_w(smem_u32(&tl->k_empty[S.ring.idx]), S.ring.phase ^ 1)) return false;
                if (elect_one()) load_k_pair(k_smem + S.ring.idx * kOperand, smem_u32(&tl->k_full[S.ring.idx]), S.it, S.cur);
                __syncwarp();
                S.ring.advance(P.n_k_stages);
                S.e = next_entry(rows, P.row_stride, S.e, g.k_top, &S.cur);
                ++S.n_issued;
                return true;
            }
            // Q goes behind the pair's first K tiles, which do not depend on the Q buffer
            if (!probe_w(smem_u32(&tl->q_empty), q_par ^ 1)) return false;
            q_par ^= 1;
            if (elect_one()) {
                const unsigned bar = smem_u32(&tl->q_full);
                mbar_arrive_expect_tx(bar, (unsigned)kOperand);
                tma_load_5d(q_smem, tq, bar, 0, S.it.qb * kBlk, S.it.h0, 0, S.it.b);  // heads h0 and h0 + 1
            }
            __syncwarp();
            S.q_due = false;
            return true;
        }
        // a V stage is free once the product computed from it is complete
        if (!probe_w(smem_u32(&tl->o_full[S.ring.idx]), S.ring.phase ^ 1)) return false;
        if (elect_one()) load_v_pair(v_smem + S.ring.idx * kOperand, smem_u32(&tl->v_full[S.ring.idx]), S.it, S.cur);
        __syncwarp();
        S.ring.advance(kVStages);
        S.e = next_entry(rows, P.row_stride, S.e, g.k_top, &S.cur);
        return true;
    };
    long long t_last = clock64();
    while (K.id < P.n_items || V.id < P.n_items) {
        const bool moved_k = step(K, true), moved_v = step(V, false);
        if (moved_k || moved_v) {
            t_last = clock64();
        } else {
            // nothing to do right now: lane 0 decides for the warp whether to go on
            int stop = 0;
            if ((threadIdx.x & 31) == 0) {
                if (*(volatile int *)&tl->abort_flag) stop = 1;
                else if (clock64() - t_last > kWaitCycles) {
                    *(volatile int *)&tl->abort_flag = 1;
                    if (atomicCAS(&g_attn_status[0], 0u, 101u) == 0u) g_attn_status[1] = blockIdx.x;
                    stop = 1;
                }
            }
            if (__shfl_sync(0xffffffffu, stop, 0)) return;
            __nanosleep(64);  // leave the issue slots to the softmax warps of this scheduler
        }
    }
}

// The two issuing roles are run by all 32 lanes of their warps, converged: the waits are
// warp-wide, one elected lane issues.

// S = [Q_0; Q_1] [K_a; K_b]^T for every kept entry.
__device__ void qk_role(const Params &P, Tail *tl, unsigned q_smem, unsigned k_smem, unsigned tmem_base) {
    const Geom &g = P.g;
    Ring ks, sb, ms;
    unsigned q_par = 0;
    const unsigned q_lo = desc_lo_sw128(q_smem, 16), k_lo = desc_lo_sw128(k_smem, 16);
    for (int id = blockIdx.x; id < P.n_items; id += gridDim.x) {
        if (!wait_w(smem_u32(&tl->m_full[ms.idx]), ms.phase, tl, 207)) return;
        const int *rows = mask_rows(tl, P, ms.idx);
        Entry cur;
        int e = next_entry(rows, P.row_stride, -1, g.k_top, &cur);
        if (e < g.k_top) {
            if (!wait_w(smem_u32(&tl->q_full), q_par, tl, 201)) return;
            q_par ^= 1;
        }
        while (e < g.k_top) {
            e = next_entry(rows, P.row_stride, e, g.k_top, &cur);  // (only "is there another entry" matters here)
            if (!wait_w(smem_u32(&tl->k_full[ks.idx]), ks.phase, tl, 202)) return;
            if (!wait_w(smem_u32(&tl->s_empty[sb.idx]), sb.phase ^ 1, tl, 203)) return;
            tc_fence_after();
            const unsigned d_tmem = tmem_base + sb.idx * 128;
            const unsigned b_lo = k_lo + ks.idx * (kOperand >> 4);
            if (elect_one()) {
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        tc_mma_bf16_split(d_tmem, q_lo + ((c * 2 * kHalfTile + k4 * 32) >> 4), kHiK,
                                          b_lo + ((c * 2 * kHalfTile + k4 * 32) >> 4), kHiK, kIdescQK, (c | k4) != 0);
                tc_commit(smem_u32(&tl->s_full[sb.idx]));
                tc_commit(smem_u32(&tl->k_empty[ks.idx]));
                if (e >= g.k_top) tc_commit(smem_u32(&tl->q_empty));  // that was the pair's last use of Q
            }
            __syncwarp();
            sb.advance(2);
            ks.advance(P.n_k_stages);
        }
        if (elect_one()) mbar_arrive(smem_u32(&tl->m_empty[ms.idx]));
        __syncwarp();
        ms.advance(kMaskSlots);
    }
}

// O = P [V_a; V_b] for every kept entry.
__device__ void pv_role(const Params &P, Tail *tl, unsigned p_smem, unsigned v_smem, unsigned tmem_base) {
    const Geom &g = P.g;
    Ring vs, ob, ms;
    unsigned p_par = 0;
    // the MN-major V tiles have their two 64-channel halves kHalfTile apart
    const unsigned p_lo = desc_lo_sw128(p_smem, 16), v_lo = desc_lo_sw128(v_smem, kHalfTile);
    for (int id = blockIdx.x; id < P.n_items; id += gridDim.x) {
        if (!wait_w(smem_u32(&tl->m_full[ms.idx]), ms.phase, tl, 208)) return;
        const int *rows = mask_rows(tl, P, ms.idx);
        Entry cur;
        int e = next_entry(rows, P.row_stride, -1, g.k_top, &cur);
        while (e < g.k_top) {
            e = next_entry(rows, P.row_stride, e, g.k_top, &cur);
            if (!wait_w(smem_u32(&tl->v_full[vs.idx]), vs.phase, tl, 205)) return;
            if (!wait_w(smem_u32(&tl->p_full), p_par, tl, 204)) return;  // also: O buffer ob has been folded
            p_par ^= 1;
            tc_fence_after();
            const unsigned d_tmem = tmem_base + 256 + ob.idx * 128;
            const unsigned b_lo = v_lo + vs.idx * (kOperand >> 4);
            if (elect_one()) {
#pragma unroll
                for (int s = 0; s < 8; ++s)  // 16 keys per step: P column half = V tile = s / 4
                    tc_mma_bf16_split(d_tmem, p_lo + (((s >> 2) * 2 * kHalfTile + (s & 3) * 32) >> 4), kHiK,
                                      b_lo + (((s >> 2) * kTile + (s & 3) * 2048) >> 4), kHiK, kIdescPV, s != 0);
                tc_commit(smem_u32(&tl->o_full[ob.idx]));  // product ready = V stage and P buffer free
            }
            __syncwarp();
            ob.advance(2);
            vs.advance(kVStages);
        }
        if (elect_one()) mbar_arrive(smem_u32(&tl->m_empty[ms.idx]));
        __syncwarp();
        ms.advance(kMaskSlots);
    }
}

// 2^x by the special-function unit (relative error about 2^-22; -inf gives 0).
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// o[0..63] = o * alpha + O, O being 64 columns of this thread's lane of a TMEM buffer.
__device__ __forceinline__ void fold_output(float *o, float alpha, unsigned taddr) {
    unsigned r[64];
    tmem_ld_32x32_issue(taddr, r);
    tmem_ld_32x32_issue(taddr + 32, r + 32);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 64; ++i) o[i] = fmaf(o[i], alpha, __uint_as_float(r[i]));
}

// Eight softmax warps. Warps w and w + 4 share the 32 TMEM lanes (query tokens) 32 (w % 4) ..: the
// first takes keys 0..31 of the token's block and output channels 0..63, the second keys 32..63
// and channels 64..127. Both read all 64 logits for the row maximum, so they only have to meet
// once per pair, to add up their partial sums (through shared memory, on an mbarrier of their own).
__device__ void softmax_role(const Params &P, Tail *tl, unsigned char *p_ptr, unsigned tmem_base, int t) {
    const Geom &g = P.g;
    const int lane = t & 31, row = t & 127, part = t >> 7, half = row >> 6, mq = row & 63, wq = row >> 5;
    const unsigned lane_off = (unsigned)(row & ~31) << 16;
    // this thread's row of the block-diagonal P operand: column half = its row of the pair
    unsigned char *p_row = p_ptr + half * 2 * kHalfTile + (row >> 3) * 1024 + (row & 7) * 128;
    const int sw = row & 7;
    const unsigned x_bar = smem_u32(&tl->x_bar[wq]);
    unsigned x_par = 0;
    int x_buf = 0;
    // publish v, meet the partner warp, return the partner's value
    auto exchange = [&](float v, float *other) -> bool {
        tl->xch[x_buf][row][part] = v;
        __syncwarp();
        if (lane == 0) mbar_arrive(x_bar);
        if (!wait(x_bar, x_par, tl, 304)) return false;
        x_par ^= 1;
        *other = tl->xch[x_buf][row][part ^ 1];
        x_buf ^= 1;
        return true;
    };
    Ring sb, ob, ms;
    for (int id = blockIdx.x; id < P.n_items; id += gridDim.x) {
        const Item it = decode_item(P, id);
        const long long tq = (long long)it.qb * kBlk + mq;
        const bool row_active = half < it.R && tq < g.T;
        if (!wait(smem_u32(&tl->m_full[ms.idx]), ms.phase, tl, 305)) return;
        const int *rows = mask_rows(tl, P, ms.idx);
        float o[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) o[i] = 0.f;
        float m = -CUDART_INF_F, l = 0.f, alpha_prev = 1.f;
        bool have_prev = false;
        Entry cur, nxt;
        int e = next_entry(rows, P.row_stride, -1, g.k_top, &cur);
        while (e < g.k_top) {
            const int e_next = next_entry(rows, P.row_stride, e, g.k_top, &nxt);  // its latency hides behind the wait
            // this token's 64 logits against its row's key block: both threads of the token read
            // all of them for the row maximum; each then exponentiates its own 32
            if (!wait(smem_u32(&tl->s_full[sb.idx]), sb.phase, tl, 301)) return;
            tc_fence_after();
            unsigned sr[64];
            const unsigned s_addr = tmem_base + sb.idx * 128 + half * 64 + lane_off;
            tmem_ld_32x32_issue(s_addr + part * 32, sr);             // own keys first
            tmem_ld_32x32_issue(s_addr + (part ^ 1) * 32, sr + 32);  // the partner's
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tl->s_empty[sb.idx]));
            sb.advance(2);
            // keys of the block this token may attend: a prefix of n_hi keys (inside T, not after it if causal)
            const int blk = half ? cur.b : cur.a;
            int n_hi = 0;
            if (blk >= 0 && row_active) {
                const long long k0 = (long long)blk * kBlk;
                long long lim = g.T - k0;
                if (g.causal) lim = min(lim, tq - k0 + 1);
                n_hi = (int)max(0ll, min(lim, (long long)kBlk));
            }
            const int n_own = n_hi - part * 32, n_oth = n_hi - (part ^ 1) * 32;  // within each half
            const bool all_keys = n_hi == kBlk;  // every block but the diagonal one and the one across T
            float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
            if (all_keys) {
#pragma unroll
                for (int i = 0; i < 64; i += 8) {
                    mx4[0] = max3(mx4[0], __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
                    mx4[1] = max3(mx4[1], __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
                    mx4[2] = max3(mx4[2], __uint_as_float(sr[i + 4]), __uint_as_float(sr[i + 5]));
                    mx4[3] = max3(mx4[3], __uint_as_float(sr[i + 6]), __uint_as_float(sr[i + 7]));
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    mx4[i & 3] = fmaxf(mx4[i & 3], i < n_own ? __uint_as_float(sr[i]) : -CUDART_INF_F);
                    mx4[i & 3] = fmaxf(mx4[i & 3], i < n_oth ? __uint_as_float(sr[32 + i]) : -CUDART_INF_F);
                }
            }
            const float m_new = fmaxf(m, fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])));
            // with no key allowed so far m_new is -inf: every p is 0 and nothing is rescaled
            const float shift = m_new == -CUDART_INF_F ? 0.f : -m_new * P.scale_log2;
            const float alpha = m_new == m ? 1.f : fast_exp2((m - m_new) * P.scale_log2);
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
            unsigned packed[16];
            if (all_keys) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(sr[i]), P.scale_log2, shift));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(sr[i + 1]), P.scale_log2, shift));
                    sum4[(i >> 1) & 3] += p0 + p1;
                    __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                    packed[i >> 1] = *reinterpret_cast<unsigned *>(&pk);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float p0 = fast_exp2(fmaf(__uint_as_float(sr[i]), P.scale_log2, shift));
                    float p1 = fast_exp2(fmaf(__uint_as_float(sr[i + 1]), P.scale_log2, shift));
                    p0 = i < n_own ? p0 : 0.f;
                    p1 = i + 1 < n_own ? p1 : 0.f;
                    sum4[(i >> 1) & 3] += p0 + p1;
                    __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                    packed[i >> 1] = *reinterpret_cast<unsigned *>(&pk);
                }
            }
            l = l * alpha + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
            m = m_new;
            // the P buffer is free, and the previous product ready, once the previous P V chain is done
            if (have_prev) {
                if (!wait(smem_u32(&tl->o_full[ob.idx]), ob.phase, tl, 302)) return;
                tc_fence_after();
            }
#pragma unroll
            for (int c = 0; c < 4; ++c)
                *reinterpret_cast<uint4 *>(p_row + (((part * 4 + c) ^ sw) << 4)) =
                    make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
            fence_async_smem();
            tc_fence_before();  // this thread's TMEM reads (the product folded last round) are done
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tl->p_full));
            if (have_prev) {
                fold_output(o, alpha_prev, tmem_base + 256 + ob.idx * 128 + part * 64 + lane_off);
                ob.advance(2);
            }
            alpha_prev = alpha;
            have_prev = true;
            e = e_next;
            cur = nxt;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&tl->m_empty[ms.idx]));
        ms.advance(kMaskSlots);
        if (have_prev) {
            if (!wait(smem_u32(&tl->o_full[ob.idx]), ob.phase, tl, 303)) return;
            tc_fence_after();
            fold_output(o, alpha_prev, tmem_base + 256 + ob.idx * 128 + part * 64 + lane_off);
            ob.advance(2);
        }
        float l_other;
        if (!exchange(l, &l_other)) return;
        if (row_active) {
            const float lt = l + l_other;
            const float inv = lt > 0.f ? 1.f / lt : 0.f;
            uint4 *dst = reinterpret_cast<uint4 *>(P.out + (((long long)it.b * g.H + it.h0 + half) * g.T + tq) * kD + part * 64);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                unsigned w[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    __nv_bfloat162 pk = __floats2bfloat162_rn(o[8 * c + 2 * j] * inv, o[8 * c + 2 * j + 1] * inv);
                    w[j] = *reinterpret_cast<unsigned *>(&pk);
                }
                dst[c] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, Params P) {  // P by value: n_k_stages is filled in here
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    // what is left behind the aligned base decides the number of K stages (the same in every thread)
    const int fixed_bytes = (int)(smem - smem_raw) + (int)sizeof(Tail) + kMaskSlots * 2 * P.row_stride * (int)sizeof(int);
    P.n_k_stages = min(kMaxKStages, (P.smem_bytes - fixed_bytes) / kOperand - kFixedOperands);
    const unsigned q_smem = smem_u32(smem), p_smem = q_smem + kOperand, v_smem = p_smem + kOperand,
                   k_smem = v_smem + kVStages * kOperand;
    Tail *tl = (Tail *)(smem + (kFixedOperands + P.n_k_stages) * kOperand);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&tl->q_full), 1);
        mbar_init(smem_u32(&tl->q_empty), 1);
        for (int i = 0; i < kMaxKStages; ++i) { mbar_init(smem_u32(&tl->k_full[i]), 1); mbar_init(smem_u32(&tl->k_empty[i]), 1); }
        for (int i = 0; i < kVStages; ++i) mbar_init(smem_u32(&tl->v_full[i]), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&tl->s_full[i]), 1); mbar_init(smem_u32(&tl->s_empty[i]), 8);
            mbar_init(smem_u32(&tl->o_full[i]), 1);
        }
        mbar_init(smem_u32(&tl->p_full), 8);
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&tl->x_bar[i]), 2);
        for (int i = 0; i < kMaskSlots; ++i) { mbar_init(smem_u32(&tl->m_full[i]), 1); mbar_init(smem_u32(&tl->m_empty[i]), 12); }
        tl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // P starts as zeros: its off-diagonal quadrants are never written again
    for (int i = threadIdx.x; i < kOperand / 16; i += kThreads)
        reinterpret_cast<uint4 *>(smem + kOperand)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    if (warp == 1) tmem_alloc_512(smem_u32(&tl->tmem_base));  // all columns: one CTA per SM
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = tl->tmem_base;

    if (warp == 0) {
        producer_role(P, &tmap_q, &tmap_k, &tmap_v, tl, q_smem, k_smem, v_smem);
    } else if (warp == 1) {
        qk_role(P, tl, q_smem, k_smem, tmem_base);
    } else if (warp == 2) {
        mask_loader_role(P, tl, lane);
    } else if (warp == 3) {
        pv_role(P, tl, p_smem, v_smem, tmem_base);
    } else {
        softmax_role(P, tl, smem + kOperand, tmem_base, (int)threadIdx.x - 128);
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

bool attn_tc_supported(const Geom &g, int dtype) {
    return dtype == STREAM_BF16 && g.d == kD && g.bq == kBlk && g.bk == kBlk && g.k_top <= kMaxKTopTc && tma_strides_ok(g);
}

stream_status launch_attn_tc(const Geom &g, const void *q, const void *k, const void *v, const int32_t *mask,
                             float scale, void *out, cudaStream_t st) {
    if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) != 0) {
        set_error("tensor-core attention kernel needs 16-byte aligned q, k, v and out");
        return STREAM_ERR_UNSUPPORTED;
    }
    CUtensorMap tq, tk, tv;
    stream_status rc = make_map5_bf16_d128(&tq, q, g.T, g.H, g.batch, g.qs_t, g.qs_h, g.qs_b, 2, "q");
    if (rc != STREAM_OK) return rc;
    rc = make_map_bf16_d128(&tk, k, g.T, g.G, g.batch, g.ks_t, g.ks_h, g.ks_b, "k");  // 4-D: 64 x 64 half tiles
    if (rc != STREAM_OK) return rc;
    rc = make_map5_bf16_d128(&tv, v, g.T, g.G, g.batch, g.ks_t, g.ks_h, g.ks_b, 1, "v");
    if (rc != STREAM_OK) return rc;
    Params P;
    P.g = g;
    P.n_pairs = (g.hpg + 1) / 2;
    const long long n_items = (long long)g.batch * g.G * g.n_qb * P.n_pairs;
    P.n_items = (int)n_items;
    P.mask = mask;
    P.out = (__nv_bfloat16 *)out;
    P.scale_log2 = scale * 1.4426950408889634f;
    const int n_sm = sm_count();
    if (n_sm <= 0) { set_error("cannot read the SM count of the current device"); return STREAM_ERR_CUDA; }
    // room for three K stages if the mask rows are short enough, else two; 1 KB of slack for the
    // alignment of the base (the kernel counts its stages from what it really gets)
    P.row_stride = (g.k_top + 3) & ~3;
    const int tail_bytes = (int)sizeof(Tail) + kMaskSlots * 2 * P.row_stride * (int)sizeof(int);
    int smem_bytes = (kFixedOperands + kMaxKStages) * kOperand + tail_bytes + 1024;
    if (smem_bytes > kMaxSmemPerCta) smem_bytes = kMaxSmemPerCta;
    if (smem_bytes < (kFixedOperands + 2) * kOperand + tail_bytes + 1024) {
        set_error("tensor-core attention kernel: k_top = %d needs more shared memory than one CTA has", g.k_top);
        return STREAM_ERR_UNSUPPORTED;
    }
    P.smem_bytes = smem_bytes;
    P.n_k_stages = 0;
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmemPerCta);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(attn_tc)");
    const int grid = (int)(n_items < n_sm ? n_items : n_sm);
    attn_tc_kernel<<<grid, kThreads, smem_bytes, st>>>(tq, tk, tv, P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "attn_tc launch");
    return STREAM_OK;
}

stream_status read_attn_status(unsigned int out[2], cudaStream_t st) {
    cudaError_t e = cudaMemcpyFromSymbolAsync(out, g_attn_status, 2 * sizeof(unsigned int), 0, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyFromSymbolAsync(attention status)");
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    return STREAM_OK;
}

}  // namespace stream
