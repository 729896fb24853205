// Tensor-core block-sparse attention for sm_100a (Eq. 2 on a Stream mask): bf16, d = 128,
// 64 x 64 blocks.
//
// One persistent CTA per SM works through "pairs": two query heads of one kv head at one query
// block. Their Q tiles are stacked into one 128-row A operand. For every mask entry e the two
// rows name one key block each (K_a, K_b, usually different); the tiles arrive by TMA (128-byte
// swizzle), stacked too, and
//     S = [Q_0; Q_1] [K_a; K_b]^T      (128 x 128, fp32 in TMEM)
// holds row 0's logits in its upper-left quadrant and row 1's in its lower-right one.
//
// Two softmax groups of four warps take a pair's entries in turn (its n-th kept entry belongs to
// group n % 2, so that a pair's arithmetic does not depend on what the CTA did before), so
// that one group's chain of waits, TMEM loads, exponentials and fences runs beside the other's.
// A thread owns one query token (TMEM lane) of its group's entries: it reads the token's 64
// logits, applies the element-level mask C, and writes P = exp2(scale (s - ref)) as bf16 into
// its row of the group's 128 x 64 A operand in shared memory. Then two chains with an
// output-lane mask,
//     O_g[lanes 0..63]   += P[rows 0..63]   V_a,      O_g[lanes 64..127] += P[rows 64..127] V_b
// (128 x 128, fp32, accumulated in TMEM per group g; V tiles MN-major), add each row's
// contribution and leave the other row's lanes alone. `ref` is a per-token reference the group keeps
// instead of the exact running maximum (bf16 P and fp32 sums keep their relative precision
// whatever the reference, as long as nothing overflows): the maximum of the token's first allowed
// logits, moved (with the token's O_g lane and sum rescaled in place) only when a logit has
// outgrown it by about 2^30 in exp2's argument, which the entry's sum of P shows. At the end of a
// pair the two groups exchange (ref, sum) per token, bring O_0 and O_1 to the common reference,
// add, normalise and store.
//
// Roles (384 threads): warp 0 TMA producer (converged, one elected lane issues; two independent
// non-blocking load streams, K with Q and V); warp 1 issues the Q K^T chains and owns TMEM; warp 3
// issues the P V chains (separate issuing warps, because the thread that issues a chain is held
// until the tensor core has taken it); warp 2 copies the pairs' mask rows from global to shared
// memory ahead of everyone else; warps 4..7 and 8..11 are the two softmax groups. Every role
// walks the same sequence of (pair, entry), read from the shared copy of the mask rows; they meet
// only on mbarriers. Every wait is bounded: on a timeout the CTA records a code in a device
// status word, raises a shared abort flag, lets its copies drain and leaves.
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
constexpr int kOperand = 2 * kTile;         // two tiles (K_a, K_b or V_a, V_b), or the 128-row Q operand
constexpr int kPBytes = 2 * kHalfTile;      // one group's P: 128 rows x 64 keys
// Stages of the two rings, out of the five operand buffers shared memory has room for beside Q
// and P (four when the mask rows are long): a V stage is held from its load until the product of
// its entry is complete, a whole softmax later, so V gets three when there are five, K two.
constexpr int kMaxKStages = 3, kMaxVStages = 3;
constexpr int kMaskSlots = 2;               // pairs whose mask rows are resident
constexpr int kMaxKTopTc = 1024;
constexpr float kLazySum = 68719476736.f;   // 2^36 = 64 * 2^30: the 64 P of an entry add up to more only if one of them exceeds 2^30 (its logit has outgrown the reference by 30 in log2 units)

// TMEM columns: S of group g at 128 g, O of group g at 256 + 128 g.
struct Tail {
    unsigned long long q_full, q_empty;
    unsigned long long k_full[kMaxKStages], k_empty[kMaxKStages], v_full[kMaxVStages], v_empty[kMaxVStages];
    // Per group g (a pair's kept entries n with n % 2 == g): logits ready / read, P published, product added.
    // o_full[g] also tells the group that its P buffer is free again.
    unsigned long long s_full[2], s_empty[2], p_full[2], o_full[2];
    unsigned long long m_full[kMaskSlots], m_empty[kMaskSlots];
    unsigned long long x_bar[4];  // the two softmax warps of a lane quarter (one per group) meet here
    unsigned int tmem_base;
    int abort_flag;
    int m_count[kMaskSlots];  // kept entries of the pair in each mask slot
};
// Dynamic shared memory: Q | P of group 0, P of group 1 | V stages | K stages | Tail | mask rows
// [kMaskSlots][2][row_stride] (-1 where a row has nothing), the operands 1024-byte aligned.
constexpr int kFixedOperands = 2;  // Q, the two P together; behind them the V stages, then the K stages
constexpr int kMaxSmemPerCta = 232448;

constexpr unsigned kIdescQK = idesc_bf16(128, 128, false);  // B = stacked K tiles, K-major
constexpr unsigned kIdescPV = idesc_bf16(128, 128, true);   // B = stacked V tiles, MN-major
constexpr unsigned kHiK = desc_hi_sw128(1024);              // every operand: 8-row (8-key) groups 1024 bytes apart

struct Params {
    Geom g;
    int n_items, n_pairs;  // pairs per kv head: ceil(hpg / 2)
    int row_stride;        // ints per resident mask row (k_top rounded up to a multiple of 4)
    int smem_bytes;        // dynamic shared memory of the launch
    int n_k_stages, n_v_stages;  // set by the kernel from what fits behind its aligned base
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
// The mask loader keeps only the kept entries of a pair, in order, at the front of the two
// resident rows and leaves their number in the Tail: entry n of a pair is (rows[n], rows[stride + n]).
__device__ __forceinline__ Entry entry_at(const int *rows, int stride, int n) {
    Entry x;
    x.a = rows[n];
    x.b = rows[stride + n];
    return x;
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
        // an entry is kept if either row has a block there; the kept ones move to the front, so that
        // the other roles index them instead of searching (their serial code is the kernel's pace)
        int cnt = 0;
        for (int base = 0; base < g.k_top; base += 32) {
            const int e = base + lane;
            int a = -1, b = -1;
            if (e < g.k_top) {
                a = __ldg(m0 + e);
                if (it.R == 2) b = __ldg(m1 + e);
            }
            const bool kept = a >= 0 || b >= 0;
            const unsigned bal = __ballot_sync(0xffffffffu, kept);
            if (kept) {
                const int pos = cnt + __popc(bal & ((1u << lane) - 1u));
                dst[pos] = a;
                dst[P.row_stride + pos] = b;
            }
            cnt += __popc(bal);
        }
        __syncwarp();
        if (lane == 0) {
            tl->m_count[ms.idx] = cnt;
            mbar_arrive(smem_u32(&tl->m_full[ms.idx]));
        }
        ms.advance(kMaskSlots);
    }
}

// One warp feeds two independent streams of TMA loads, the K tiles (with each pair's Q tiles)
// and the V tiles, each as far ahead as its ring of stages allows. It never blocks on one stream
// while the other could move: every step probes its barrier without waiting. The warp runs
// converged (lane 0's probe result is broadcast) and one elected lane issues.
struct LoadStream {
    int id;            // pair being walked
    int e;             // current entry (n = pair exhausted), -2 = pair not opened yet
    int n;             // kept entries of the pair
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
            S.n = tl->m_count[S.ms.idx];
            S.e = 0;
            if (S.n > 0) S.cur = entry_at(rows, P.row_stride, 0);
            S.q_due = is_k && S.n > 0;  // (a pair with nothing kept: only the softmax warps act)
            S.n_issued = 0;
            return true;
        }
        if (S.e >= S.n && !S.q_due) {  // pair exhausted: give its mask rows back, go to the next one
            if (elect_one()) mbar_arrive(smem_u32(&tl->m_empty[S.ms.idx]));
            __syncwarp();
            S.ms.advance(kMaskSlots);
            S.id += gridDim.x;
            S.e = -2;
            return true;
        }
        if (is_k) {
            if (S.e < S.n && !(S.q_due && S.n_issued > 0)) {
                // a K stage is free once the logits computed from it are complete
                if (!probe_w(smem_u32(&tl->k_empty[S.ring.idx]), S.ring.phase ^ 1)) return false;
                if (elect_one()) load_k_pair(k_smem + S.ring.idx * kOperand, smem_u32(&tl->k_full[S.ring.idx]), S.it, S.cur);
                __syncwarp();
                S.ring.advance(P.n_k_stages);
                if (++S.e < S.n) S.cur = entry_at(rows, P.row_stride, S.e);
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
        if (!probe_w(smem_u32(&tl->v_empty[S.ring.idx]), S.ring.phase ^ 1)) return false;
        if (elect_one()) load_v_pair(v_smem + S.ring.idx * kOperand, smem_u32(&tl->v_full[S.ring.idx]), S.it, S.cur);
        __syncwarp();
        S.ring.advance(P.n_v_stages);
        if (++S.e < S.n) S.cur = entry_at(rows, P.row_stride, S.e);
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
            __nanosleep(200);  // leave the issue slots to the softmax warps of this scheduler
        }
    }
}

// The two issuing roles are run by all 32 lanes of their warps, converged: the waits are
// warp-wide, one elected lane issues.

// S_g = [Q_0; Q_1] [K_a; K_b]^T for every kept entry (g = the entry's number within its pair % 2).
__device__ void qk_role(const Params &P, Tail *tl, unsigned q_smem, unsigned k_smem, unsigned tmem_base) {
    Ring ks, ms;
    unsigned cnt[2] = {0, 0};  // entries each group has had over the whole kernel
    unsigned q_par = 0;
    const unsigned q_lo = desc_lo_sw128(q_smem, 16), k_lo = desc_lo_sw128(k_smem, 16);
    for (int id = blockIdx.x; id < P.n_items; id += gridDim.x) {
        if (!wait_w(smem_u32(&tl->m_full[ms.idx]), ms.phase, tl, 207)) return;
        const int n_entries = tl->m_count[ms.idx];  // the issuers need no more than the count
        if (n_entries > 0) {
            if (!wait_w(smem_u32(&tl->q_full), q_par, tl, 201)) return;
            q_par ^= 1;
        }
        for (int i = 0; i < n_entries; ++i) {
            if (!wait_w(smem_u32(&tl->k_full[ks.idx]), ks.phase, tl, 202)) return;
            const unsigned gi = (unsigned)(i & 1), use = cnt[gi]++;  // entry i of a pair belongs to group i % 2
            if (!wait_w(smem_u32(&tl->s_empty[gi]), (use & 1u) ^ 1u, tl, 203)) return;
            tc_fence_after();
            const unsigned d_tmem = tmem_base + gi * 128;
            const unsigned b_lo = k_lo + ks.idx * (kOperand >> 4);
            if (elect_one()) {
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        tc_mma_bf16_split(d_tmem, q_lo + ((c * 2 * kHalfTile + k4 * 32) >> 4), kHiK,
                                          b_lo + ((c * 2 * kHalfTile + k4 * 32) >> 4), kHiK, kIdescQK, (c | k4) != 0);
                tc_commit(smem_u32(&tl->s_full[gi]));
                tc_commit(smem_u32(&tl->k_empty[ks.idx]));
                if (i + 1 == n_entries) tc_commit(smem_u32(&tl->q_empty));  // that was the pair's last use of Q
            }
            __syncwarp();
            ks.advance(P.n_k_stages);
        }
        if (elect_one()) mbar_arrive(smem_u32(&tl->m_empty[ms.idx]));
        __syncwarp();
        ms.advance(kMaskSlots);
    }
}

// O_g (+)= P_g [V_a; V_b] for every kept entry; a group's first entry of a pair starts its O afresh.
__device__ void pv_role(const Params &P, Tail *tl, unsigned p_smem, unsigned v_smem, unsigned tmem_base) {
    Ring vs, ms;  // vs: the entry's V stage
    unsigned cnt[2] = {0, 0};  // entries each group has had over the whole kernel
    // the MN-major V tiles have their two 64-channel halves kHalfTile apart
    const unsigned p_lo = desc_lo_sw128(p_smem, 16), v_lo = desc_lo_sw128(v_smem, kHalfTile);
    for (int id = blockIdx.x; id < P.n_items; id += gridDim.x) {
        if (!wait_w(smem_u32(&tl->m_full[ms.idx]), ms.phase, tl, 208)) return;
        const int n_entries = tl->m_count[ms.idx];
        unsigned fresh = 3u;  // bit g: group g has not added anything for this pair yet
        for (int i = 0; i < n_entries; ++i) {
            if (!wait_w(smem_u32(&tl->v_full[vs.idx]), vs.phase, tl, 205)) return;
            const unsigned gi = (unsigned)(i & 1), use = cnt[gi]++;  // group = O buffer of the entry
            if (!wait_w(smem_u32(&tl->p_full[gi]), use & 1u, tl, 204)) return;  // also: O_g rescaled if it had to be
            tc_fence_after();
            const unsigned d_tmem = tmem_base + 256 + gi * 128;
            const unsigned a_lo = p_lo + gi * (kPBytes >> 4), b_lo = v_lo + vs.idx * (kOperand >> 4);
            const unsigned keep = ((fresh >> gi) & 1u) ^ 1u;
            fresh &= ~(1u << gi);
            if (elect_one()) {
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {  // row `tile` of the pair: its P rows, its V tile, its lanes
                    const unsigned lo_off = tile ? 0xFFFFFFFFu : 0u, hi_off = tile ? 0u : 0xFFFFFFFFu;
#pragma unroll
                    for (int s4 = 0; s4 < 4; ++s4)  // 16 keys per step
                        tc_mma_bf16_split_masked(d_tmem, a_lo + ((s4 * 32) >> 4), kHiK, b_lo + ((tile * kTile + s4 * 2048) >> 4),
                                                 kHiK, kIdescPV, s4 != 0 ? 1u : keep, lo_off, lo_off, hi_off, hi_off);
                }
                tc_commit(smem_u32(&tl->o_full[gi]));  // product added: the group's P buffer is free
                tc_commit(smem_u32(&tl->v_empty[vs.idx]));
            }
            __syncwarp();
            vs.advance(P.n_v_stages);
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

// Multiplies 128 fp32 columns of this thread's TMEM lane by f, in place (every lane of the warp
// takes part; lanes that need no change pass f = 1).
__device__ __forceinline__ void rescale_lane(unsigned taddr, float f) {
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
        unsigned r[32];
        tmem_ld_32x32_issue(taddr + c * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
        tmem_st_32x32_issue(taddr + c * 32, r);
    }
    tmem_st_wait();
}

// One softmax group: four warps, thread = query token (TMEM lane) `row` of the pair, for the
// entries n with n % 2 == grp (n numbers the kept entries of each pair, as in every role).
// The waits are warp-wide (same answer in every lane), so the warp stays converged for the
// warp-collective TMEM loads and stores and leaves together if the CTA aborts.
__device__ void softmax_role(const Params &P, Tail *tl, unsigned char *p_ptr, unsigned tmem_base, int t) {
    const Geom &g = P.g;
    const int lane = t & 31, row = t & 127, grp = t >> 7, half = row >> 6, mq = row & 63, wq = row >> 5;
    const unsigned lane_off = (unsigned)(row & ~31) << 16;
    // this thread's row of its group's P operand, and the same row in the other group's: the two
    // exchange a few bytes there at the end of a pair
    const int row_off = (row >> 3) * 1024 + (row & 7) * 128;
    unsigned char *p_row = p_ptr + grp * kPBytes + row_off;
    const unsigned char *p_row_other = p_ptr + (grp ^ 1) * kPBytes + row_off;
    const int sw = row & 7;
    const unsigned s_full = smem_u32(&tl->s_full[grp]), s_empty = smem_u32(&tl->s_empty[grp]),
                   p_full = smem_u32(&tl->p_full[grp]), o_full = smem_u32(&tl->o_full[grp]), x_bar = smem_u32(&tl->x_bar[wq]);
    const unsigned s_addr = tmem_base + grp * 128 + half * 64 + lane_off;
    const unsigned o_own = tmem_base + 256 + grp * 128 + lane_off, o_other = tmem_base + 256 + (grp ^ 1) * 128 + lane_off;
    unsigned s_par = 0, o_par = 0, x_par = 0;
    Ring ms;
    for (int id = blockIdx.x; id < P.n_items; id += gridDim.x) {
        const Item it = decode_item(P, id);
        const long long tq = (long long)it.qb * kBlk + mq;
        const bool row_active = half < it.R && tq < g.T;
        if (!wait_w(smem_u32(&tl->m_full[ms.idx]), ms.phase, tl, 305)) return;
        const int *rows = mask_rows(tl, P, ms.idx);
        float ref = -CUDART_INF_F, l = 0.f;
        bool ref_open = true;  // some token of this warp has no reference yet (the same in every lane)
        bool pending = false;  // a P V chain of this group and pair may still be running
        const int n_entries = tl->m_count[ms.idx];
        const int *my_row = rows + half * P.row_stride;  // this token's row of the pair
        for (int n = grp; n < n_entries; n += 2) {  // entry n of a pair belongs to group n % 2
            // the token's 64 logits against its row's key block
            if (!wait_w(s_full, s_par, tl, 301)) return;
            s_par ^= 1;
            tc_fence_after();
            unsigned sr[64];
            tmem_ld_32x32_issue(s_addr, sr);
            tmem_ld_32x32_issue(s_addr + 32, sr + 32);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty);
            // keys of the block this token may attend: a prefix of n_hi keys (inside T, not after it if causal)
            const int blk = my_row[n];
            int n_hi = 0;
            if (blk >= 0 && row_active) {
                const long long k0 = (long long)blk * kBlk;
                long long lim = g.T - k0;
                if (g.causal) lim = min(lim, tq - k0 + 1);
                n_hi = (int)max(0ll, min(lim, (long long)kBlk));
            }
            const bool all_keys = n_hi == kBlk;  // every block but the diagonal one and the one across T
            // P = exp2(scale (s - ref)) under the token's current reference, their sum, the packed row.
            // No reference yet (+inf shift: any allowed logit then gives +inf) or a logit that has
            // outgrown the reference by more than kLazyLog2 both show in the sum of the 64 P, which
            // is needed anyway: the maximum itself is only taken when that happens.
            unsigned packed[32];
            float esum;
            auto make_p = [&](float shift) {
                float sum4[4] = {0.f, 0.f, 0.f, 0.f};
                if (all_keys) {
#pragma unroll
                    for (int i = 0; i < 64; i += 2) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sr[i]), P.scale_log2, shift));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sr[i + 1]), P.scale_log2, shift));
                        sum4[(i >> 1) & 3] += p0 + p1;
                        __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                        packed[i >> 1] = *reinterpret_cast<unsigned *>(&pk);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 64; i += 2) {
                        float p0 = fast_exp2(fmaf(__uint_as_float(sr[i]), P.scale_log2, shift));
                        float p1 = fast_exp2(fmaf(__uint_as_float(sr[i + 1]), P.scale_log2, shift));
                        p0 = i < n_hi ? p0 : 0.f;
                        p1 = i + 1 < n_hi ? p1 : 0.f;
                        sum4[(i >> 1) & 3] += p0 + p1;
                        __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                        packed[i >> 1] = *reinterpret_cast<unsigned *>(&pk);
                    }
                }
                esum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            };
            auto masked_max = [&]() {
                float x[64];
#pragma unroll
                for (int i = 0; i < 64; ++i) x[i] = i < n_hi ? __uint_as_float(sr[i]) : -CUDART_INF_F;
                return max_of_64(x);
            };
            // the token's first allowed logits set its reference (once per pair)
            if (ref_open && __any_sync(0xffffffffu, ref == -CUDART_INF_F && n_hi > 0)) {
                const float mx = masked_max();
                if (ref == -CUDART_INF_F) ref = mx;
                ref_open = __any_sync(0xffffffffu, ref == -CUDART_INF_F);
            }
            make_p(ref == -CUDART_INF_F ? 0.f : -ref * P.scale_log2);
            const bool redo = !(esum <= kLazySum);
            // this group's previous chain of the pair must be done before its P buffer is rewritten
            // or its O lane rescaled
            if (pending) {
                if (!wait_w(o_full, o_par, tl, 302)) return;
                o_par ^= 1;
                tc_fence_after();
            }
            if (__any_sync(0xffffffffu, redo)) {  // rare: a logit has outgrown the token's reference
                const float mx = masked_max();
                float f = 1.f;
                if (redo) {
                    f = fast_exp2((ref - mx) * P.scale_log2);
                    ref = mx;
                }
                // what the group has accumulated for this token is brought to the new reference
                rescale_lane(o_own, f);
                l *= f;
                if (redo) make_p(-ref * P.scale_log2);
            }
            l += esum;
#pragma unroll
            for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4 *>(p_row + ((c ^ sw) << 4)) =
                    make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
            fence_async_smem();
            tc_fence_before();  // the rescaled O lane, if any, is in place
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);
            pending = true;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&tl->m_empty[ms.idx]));
        ms.advance(kMaskSlots);
        // End of the pair: bring the two groups' sums to a common reference and store.
        if (pending) {
            if (!wait_w(o_full, o_par, tl, 303)) return;
            o_par ^= 1;
            tc_fence_after();
        }
        *reinterpret_cast<float2 *>(p_row) = make_float2(ref, l);  // the P row is free: use it as mailbox
        __syncwarp();
        if (lane == 0) mbar_arrive(x_bar);
        if (!wait_w(x_bar, x_par, tl, 304)) return;
        x_par ^= 1;
        tc_fence_after();  // the other group's last chain is complete too
        const float2 oth = *reinterpret_cast<const float2 *>(p_row_other);
        const float top = fmaxf(ref, oth.x);
        const float f_own = ref == -CUDART_INF_F ? 0.f : fast_exp2((ref - top) * P.scale_log2);
        const float f_oth = oth.x == -CUDART_INF_F ? 0.f : fast_exp2((oth.x - top) * P.scale_log2);
        const float total = l * f_own + oth.y * f_oth;
        const float inv = total > 0.f ? 1.f / total : 0.f;
        const float w_own = f_own * inv, w_oth = f_oth * inv;
        // this group stores channels 64 grp .. 64 grp + 63 of every token
        uint4 out_words[8];
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            unsigned ra[32], rb[32];
            tmem_ld_32x32_issue(o_own + grp * 64 + c * 32, ra);
            tmem_ld_32x32_issue(o_other + grp * 64 + c * 32, rb);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                unsigned w[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = 8 * j + 2 * u;
                    // a group without entries in this pair holds stale numbers: weight 0 means "leave out"
                    const float a0 = w_own != 0.f ? __uint_as_float(ra[i]) * w_own : 0.f;
                    const float a1 = w_own != 0.f ? __uint_as_float(ra[i + 1]) * w_own : 0.f;
                    const float v0 = w_oth != 0.f ? fmaf(__uint_as_float(rb[i]), w_oth, a0) : a0;
                    const float v1 = w_oth != 0.f ? fmaf(__uint_as_float(rb[i + 1]), w_oth, a1) : a1;
                    __nv_bfloat162 pk = __floats2bfloat162_rn(v0, v1);
                    w[u] = *reinterpret_cast<unsigned *>(&pk);
                }
                out_words[c * 4 + j] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        // second meeting: both groups have read both O buffers and both mailboxes
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(x_bar);
        if (!wait_w(x_bar, x_par, tl, 306)) return;
        x_par ^= 1;
        if (row_active) {
            uint4 *dst = reinterpret_cast<uint4 *>(P.out + (((long long)it.b * g.H + it.h0 + half) * g.T + tq) * kD + grp * 64);
#pragma unroll
            for (int c = 0; c < 8; ++c) dst[c] = out_words[c];
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, Params P) {  // P by value: n_k_stages is filled in here
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    // what is left behind the aligned base decides the number of V and K stages (the same in every thread)
    const int fixed_bytes = (int)(smem - smem_raw) + (int)sizeof(Tail) + kMaskSlots * 2 * P.row_stride * (int)sizeof(int);
    const int n_rings = (P.smem_bytes - fixed_bytes) / kOperand - kFixedOperands;  // buffers for the two rings: 4 or 5
    P.n_v_stages = n_rings >= 5 ? 3 : 2;
    P.n_k_stages = min(kMaxKStages, n_rings - P.n_v_stages);
    const unsigned q_smem = smem_u32(smem), p_smem = q_smem + kOperand, v_smem = p_smem + 2 * kPBytes,
                   k_smem = v_smem + P.n_v_stages * kOperand;
    Tail *tl = (Tail *)(smem + (kFixedOperands + P.n_v_stages + P.n_k_stages) * kOperand);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&tl->q_full), 1);
        mbar_init(smem_u32(&tl->q_empty), 1);
        for (int i = 0; i < kMaxKStages; ++i) { mbar_init(smem_u32(&tl->k_full[i]), 1); mbar_init(smem_u32(&tl->k_empty[i]), 1); }
        for (int i = 0; i < kMaxVStages; ++i) { mbar_init(smem_u32(&tl->v_full[i]), 1); mbar_init(smem_u32(&tl->v_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&tl->s_full[i]), 1); mbar_init(smem_u32(&tl->s_empty[i]), 4);
            mbar_init(smem_u32(&tl->p_full[i]), 4); mbar_init(smem_u32(&tl->o_full[i]), 1);
        }
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&tl->x_bar[i]), 2);
        for (int i = 0; i < kMaskSlots; ++i) { mbar_init(smem_u32(&tl->m_full[i]), 1); mbar_init(smem_u32(&tl->m_empty[i]), 12); }
        tl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
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
    // room for five ring buffers (three V, two K) if the mask rows are short enough, else four; 1 KB of slack for the
    // alignment of the base (the kernel counts its stages from what it really gets)
    P.row_stride = (g.k_top + 3) & ~3;
    const int tail_bytes = (int)sizeof(Tail) + kMaskSlots * 2 * P.row_stride * (int)sizeof(int);
    int smem_bytes = (kFixedOperands + 5) * kOperand + tail_bytes + 1024;
    if (smem_bytes > kMaxSmemPerCta) smem_bytes = kMaxSmemPerCta;
    if (smem_bytes < (kFixedOperands + 4) * kOperand + tail_bytes + 1024) {
        set_error("tensor-core attention kernel: k_top = %d needs more shared memory than one CTA has", g.k_top);
        return STREAM_ERR_UNSUPPORTED;
    }
    P.smem_bytes = smem_bytes;
    P.n_k_stages = P.n_v_stages = 0;
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
