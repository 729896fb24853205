// Tensor-core Stream mask kernel for sm_100a: bf16, d = 128, 64 x 64 blocks, k_top <= 32.
//
// One persistent CTA per SM works through "groups": up to four query heads of one kv head at
// one query block. Their Q tiles stay in shared memory for the whole hierarchy (Algorithm 2).
// Candidate key blocks are fetched by TMA (128-byte swizzle) two at a time into a ring of
// stages; one tcgen05.mma chain per (stage, row) computes K_pair (128 x 128) x Q_row^T (128 x 64)
// into a 64-column TMEM slot; four epilogue warps reduce the slot to the two masked tile maxima
// (Eq. 4 under C). There are two such groups of four, each serving one of every issuing warp's
// two slots: the fixed cost of a hand-over (wait, fences, arrive) is larger than the reduction
// itself, and one group alone would be the longest stage of the pipeline. A controller warp keeps
// each row's nodes in registers, ranks the 2k branch scores (higher score, then lower block
// index), compacts the survivors with ballots and publishes the next level's fetch list. The
// first level's representatives are the same for every row of a group, so one fetched stage
// serves all its rows; from the second level on a left branch inherits its parent's score and
// only right branches are fetched. With several k per call a group runs the hierarchy once per
// k on the same Q tiles and fetches only blocks whose score it does not have yet.
//
// Roles (512 threads, the last warp idle): warps 0 and 14 TMA producers (even and odd stage
// buffers; warp 0 also brings the Q tiles), warps 1, 3, 12, 13 MMA issuers (warp 1 owns TMEM),
// warp 2 controller, warps 4..7 and 8..11 the two epilogue groups (TMEM lane quarter = warp % 4). All roles walk the same fixed unit order (level 1: stage-major,
// row-minor; later levels: row-major), synchronised by mbarriers only. Every wait is bounded: on
// a timeout the CTA records an error code in the workspace header, raises a shared abort flag,
// drains its own copies and leaves.
#include <math_constants.h>

#include "tc_common.cuh"

namespace stream {
namespace {

using namespace tc;

constexpr int kThreads = 512;
constexpr int kEpiGroups = 2;  // group g reduces the chains that land in slot g of their issuing warp
constexpr int kMmaWarps = 4;   // warps 1, 3, 12, 13 take the stages in turn
constexpr int kR = 4;          // rows (query heads) per group
constexpr int kStages = 4;     // K-pair stages
constexpr int kSlots = 8;      // TMEM accumulator slots of 64 fp32 columns
constexpr int kBlk = 64, kD = 128;
constexpr int kHalfTile = kBlk * 128;          // 64 rows x 128 bytes (one 64-channel half)
constexpr int kStageBytes = 4 * kHalfTile;     // [2 channel halves][2 tiles]
constexpr int kQBytes = 2 * kR * kHalfTile;    // [2 channel halves][kR rows]
constexpr int kMaxJobs = 64;
constexpr int kProducers = 2;     // warps 0 and 14: producer p fills the stage buffers b with b % 2 == p
constexpr int kListReaders = kProducers + kMmaWarps + 4 * kEpiGroups;  // producer, MMA and epilogue warps
// A parity wait only means something to a thread that saw the phase before it complete, and an
// arrival only if it cannot come a phase early. So every stage buffer and every TMEM slot
// belongs to one issuing warp: stage s of the kernel's whole sequence goes, with all its chains,
// to warp s % kMmaWarps and lands in buffer s % kStages (the same number), and a warp's chains
// alternate between its own two slots. The other issuing warps touch none of its barriers.
static_assert(kStages == kMmaWarps, "a stage buffer must always meet the same issuing warp");
static_assert(kSlots == 2 * kMmaWarps, "two private TMEM slots per issuing warp");

struct Tail {
    unsigned long long full[kStages], empty[kStages], tmem_full[kSlots], tmem_empty[kSlots];
    unsigned long long q_full, jobs_ready[kR + 1], scores_done[kR];
    // jobs_ack[i]: every reader of list i (the producer, the MMA warps, the epilogue warps) has
    // taken what it needs from n_jobs[i], jobs_blk[i] and, for i = kR, the group record; the
    // controller waits for it before it writes them again. Without it a warp with nothing to do
    // in a short list could still be about to read it when the next one is written, or fall two
    // phases behind jobs_ready[i].
    unsigned long long jobs_ack[kR + 1];
    unsigned int tmem_base;
    int abort_flag;
    int grp_id, grp_b, grp_kvh, grp_qb, grp_h0, grp_R;
    int grp_levels;  // levels of this group's rows (they share the query block, hence k)
    int grp_new_q;   // 0: another pass over the same rows (several k), the Q tiles are already there
    int n_jobs[kR + 1];
    int jobs_blk[kR + 1][kMaxJobs];
    float part[kR][kMaxJobs][2];
    int node_f[32], node_l[32];
    float node_s[32];
};
constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + (int)sizeof(Tail) + 1024;

// Bounded wait that reports into the workspace header; false means the CTA is aborting.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, Tail *tl, WorkspaceHeader *ws, unsigned code) {
    return mbar_wait_bounded(bar, parity, &tl->abort_flag, &ws->error, &ws->error_info, code);
}

// The same for a whole converged warp (all lanes get the same answer).
__device__ __forceinline__ bool mbar_wait_w(unsigned bar, unsigned parity, Tail *tl, WorkspaceHeader *ws, unsigned code) {
    return mbar_wait_warp(bar, parity, &tl->abort_flag, &ws->error, &ws->error_info, code);
}

// K-major, 128-byte-swizzled operands with 8-row groups 1024 bytes apart: high descriptor word.
constexpr unsigned kDescHi = desc_hi_sw128(1024);

// D fp32, A and B bf16, both K-major, M = 128, N = 64.
constexpr unsigned kIdesc = idesc_bf16(128, 64, false);

struct Params {
    Geom g;
    int n_groups, n_chunks;
    int32_t *mask;
    float *score;
    WorkspaceHeader *ws;
    // Several sparsity constants in one launch: a group runs the hierarchy once per k, with its Q
    // tiles loaded once, and writes mask slab `pass`. A tile's score does not depend on k, so the
    // controller remembers every (row, block) score of the group in `cache` (one entry per row
    // and key block for each CTA: {group tag, score}) and only lists blocks no earlier pass scored.
    MultiK mk;                      // n = 0: one pass with the geometry's k
    unsigned long long *cache;      // [gridDim.x][kR][N_k], zeroed before the launch; NULL = no sharing
    long long slab;                 // elements between two mask slabs
};

__device__ __forceinline__ unsigned long long cache_pack(unsigned tag, float s) {
    return ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(s);
}

// ----------------------------------------------------------------------------------------------
// Roles
// ----------------------------------------------------------------------------------------------
// Run by all 32 lanes of a producer warp, converged (warp-wide waits, one elected lane issues): a
// single diverged lane issues TMA copies several times more slowly. Two producers share the
// stages by buffer parity: one alone is busy more than half of the time with the four copies and
// the barrier arm of a stage, and the issuing warps then wait for data.
__device__ void producer_role(const Params &P, const CUtensorMap *tq, const CUtensorMap *tk, Tail *tl, unsigned q_smem,
                              unsigned k_smem, int which) {
    Ring st;
    unsigned grp_par = 0, jr_par[kR] = {0, 0, 0, 0};
    unsigned long long fetched = 0;  // tiles this warp has asked TMA for
    for (;;) {
        if (!mbar_wait_w(smem_u32(&tl->jobs_ready[kR]), grp_par, tl, P.ws, 101)) return;
        grp_par ^= 1;
        if (tl->grp_id < 0) {
            if (elect_one()) atomicAdd(&P.ws->tiles_fetched, fetched);
            return;
        }
        const int b = tl->grp_b, kvh = tl->grp_kvh, qb = tl->grp_qb, h0 = tl->grp_h0, R = tl->grp_R;
        const int levels = tl->grp_levels;
        // Q tiles of the group's rows (previous group's MMAs are all complete by now)
        if (which == 0 && tl->grp_new_q && elect_one()) {
            mbar_arrive_expect_tx(smem_u32(&tl->q_full), (unsigned)(R * 2 * kHalfTile));
            for (int r = 0; r < R; ++r)
                for (int c = 0; c < 2; ++c)
                    tma_load_4d(q_smem + (c * kR + r) * kHalfTile, tq, smem_u32(&tl->q_full), c * 64, qb * kBlk, h0 + r, b);
        }
        if (which == 0 && tl->grp_new_q) fetched += (unsigned)R;
        __syncwarp();
        for (int level = 0; level < levels; ++level) {
            const int lists = level == 0 ? 1 : R;
            for (int x = 0; x < lists; ++x) {
                const int li = level == 0 ? kR : x;
                if (level > 0) {
                    if (!mbar_wait_w(smem_u32(&tl->jobs_ready[x]), jr_par[x], tl, P.ws, 102)) return;
                    jr_par[x] ^= 1;
                }
                const int n = tl->n_jobs[li];
                for (int j = 0; j < n; j += 2) {
                    if ((st.idx & (kProducers - 1)) != which) { st.advance(kStages); continue; }  // the other producer's buffer
                    if (!mbar_wait_w(smem_u32(&tl->empty[st.idx]), st.phase ^ 1, tl, P.ws, 103)) return;
                    const int two = (j + 1 < n);
                    fetched += 1u + (unsigned)two;
                    const int blk0 = tl->jobs_blk[li][j], blk1 = two ? tl->jobs_blk[li][j + 1] : 0;
                    if (elect_one()) {
                        const unsigned bar = smem_u32(&tl->full[st.idx]);
                        const unsigned dst = k_smem + st.idx * kStageBytes;
                        mbar_arrive_expect_tx(bar, (unsigned)((two ? 4 : 2) * kHalfTile));
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            tma_load_4d(dst + c * 2 * kHalfTile, tk, bar, c * 64, blk0 * kBlk, kvh, b);
                            if (two) tma_load_4d(dst + (c * 2 + 1) * kHalfTile, tk, bar, c * 64, blk1 * kBlk, kvh, b);
                        }
                    }
                    __syncwarp();
                    st.advance(kStages);
                }
                if (elect_one()) mbar_arrive(smem_u32(&tl->jobs_ack[li]));  // done reading this list
                __syncwarp();
            }
        }
    }
}

// kMmaWarps warps take the stages in turn (stage s belongs, with all its chains, to warp
// s % kMmaWarps): the waits, commits and bookkeeping between two chains of one warp take several
// times longer than the tensor core needs for a chain, so one issuing warp would leave it idle
// most of the time. All issuing warps walk the same unit order; each is run by all 32 lanes,
// converged: warp-wide waits, one elected lane issues.
//
// Which of the owner's two TMEM slots a chain lands in is a fixed function of its place in the
// unit order, so that the issuing warp and the epilogue groups agree on it without counting each
// other's chains: on the first level chain r of a stage goes to slot r % 2, later (one chain per
// stage) the chain of stage s goes to slot (s / kMmaWarps) % 2. Both sides keep one phase bit per
// slot they use.
__device__ __forceinline__ int chain_slot(int level, int r, unsigned stage) {
    return level == 0 ? (r & 1) : (int)((stage / kMmaWarps) & 1u);
}

__device__ void mma_role(const Params &P, Tail *tl, unsigned q_smem, unsigned k_smem, unsigned tmem_base, int which) {
    unsigned grp_par = 0, q_par = 0, jr_par[kR] = {0, 0, 0, 0};
    unsigned stage_seq = 0;   // stages so far, over the whole kernel (the same in every role)
    unsigned slot_par = 0;    // bit i: phase of the next use of this warp's slot i
    const unsigned q_lo = desc_lo_sw128(q_smem, 16);
    const int sidx = which;   // this warp's stage buffer: stage s lands in buffer s % kStages
    const unsigned a_lo = desc_lo_sw128(k_smem + sidx * kStageBytes, 16);
    for (;;) {
        if (!mbar_wait_w(smem_u32(&tl->jobs_ready[kR]), grp_par, tl, P.ws, 201)) return;
        grp_par ^= 1;
        if (tl->grp_id < 0) return;
        const int R = tl->grp_R, levels = tl->grp_levels;
        if (tl->grp_new_q) {
            if (!mbar_wait_w(smem_u32(&tl->q_full), q_par, tl, P.ws, 202)) return;
            q_par ^= 1;
        }
        for (int level = 0; level < levels; ++level) {
            const int lists = level == 0 ? 1 : R;
            for (int x = 0; x < lists; ++x) {
                const int li = level == 0 ? kR : x;
                if (level > 0) {
                    if (!mbar_wait_w(smem_u32(&tl->jobs_ready[x]), jr_par[x], tl, P.ws, 203)) return;
                    jr_par[x] ^= 1;
                }
                const unsigned n_st = (unsigned)(tl->n_jobs[li] + 1) >> 1;  // stages of this list
                __syncwarp();
                if (elect_one()) mbar_arrive(smem_u32(&tl->jobs_ack[li]));  // the count is all this role reads
                __syncwarp();
                const int r0 = level == 0 ? 0 : x, r1 = level == 0 ? R : x + 1;
                const unsigned s_end = stage_seq + n_st;
                // this warp's stages of the list: s = which (mod kMmaWarps)
                for (unsigned s = stage_seq + (((unsigned)which - stage_seq) & (kMmaWarps - 1)); s < s_end; s += kMmaWarps) {
                    if (!mbar_wait_w(smem_u32(&tl->full[sidx]), (s / kStages) & 1u, tl, P.ws, 204)) return;
                    for (int r = r0; r < r1; ++r) {
                        const int sl = chain_slot(level, r, s);
                        const int slot = 2 * which + sl;
                        if (!mbar_wait_w(smem_u32(&tl->tmem_empty[slot]), ((slot_par >> sl) & 1u) ^ 1u, tl, P.ws, 205)) return;
                        slot_par ^= 1u << sl;
                        tc_fence_after();
                        const unsigned d_tmem = tmem_base + slot * 64;
                        const unsigned b_lo = q_lo + r * (kHalfTile >> 4);
                        if (elect_one()) {
#pragma unroll
                            for (int c = 0; c < 2; ++c)
#pragma unroll
                                for (int k4 = 0; k4 < 4; ++k4)
                                    tc_mma_bf16_split(d_tmem, a_lo + ((c * 2 * kHalfTile + k4 * 32) >> 4), kDescHi,
                                                      b_lo + ((c * kR * kHalfTile + k4 * 32) >> 4), kDescHi, kIdesc, (c | k4) != 0);
                            tc_commit(smem_u32(&tl->tmem_full[slot]));
                            // the stage is free once its last chain has read it (a commit covers all
                            // earlier instructions of this thread)
                            if (r + 1 == r1) tc_commit(smem_u32(&tl->empty[sidx]));
                        }
                        __syncwarp();
                    }
                }
                stage_seq = s_end;
            }
        }
    }
}

// One epilogue group (four warps, one per TMEM lane quarter). Group `grp` waits for and reduces
// the chains that land in slot `grp` of their issuing warp (chain_slot): a slot's barriers are
// then used by one group only, which sees every phase of them. It steps over the other group's
// chains without looking at them: the bookkeeping of a warp is serial code, and what it spends
// there it cannot spend reducing.
__device__ void epilogue_role(const Params &P, Tail *tl, unsigned tmem_base, int wq, int grp, int lane) {
    const Geom &g = P.g;
    unsigned grp_par = 0, jr_par[kR] = {0, 0, 0, 0};
    unsigned stage_seq = 0;
    unsigned full_par = 0;  // bit w: phase of the next use of issuing warp w's slot `grp`
    const int tile = wq >> 1;                // which tile of the pair this warp's lanes hold
    const int key = (wq & 1) * 32 + lane;    // key index inside the tile
    const unsigned t_lane = tmem_base + ((unsigned)(wq * 32) << 16) + grp * 64;
    for (;;) {
        if (!mbar_wait(smem_u32(&tl->jobs_ready[kR]), grp_par, tl, P.ws, 301)) return;
        grp_par ^= 1;
        if (tl->grp_id < 0) return;
        const int R = tl->grp_R, qb = tl->grp_qb, levels = tl->grp_levels;
        const long long rem_q = g.T - (long long)qb * kBlk;
        const int m_lim = rem_q < kBlk ? (int)rem_q : kBlk;  // query tokens of this block inside T
        // One chain of this group: stage s, row r, this warp's tile at position c of list li.
        auto reduce = [&](unsigned s, int r, int li, int c, int n) -> bool {
            const unsigned owner = s & (kMmaWarps - 1);
            const unsigned slot = 2 * owner + grp;
            if (!mbar_wait(smem_u32(&tl->tmem_full[slot]), (full_par >> owner) & 1u, tl, P.ws, 303)) return false;
            full_par ^= 1u << owner;
            tc_fence_after();
            if (c < n) {
                const int blk = tl->jobs_blk[li][c];
                float v[64];
                const unsigned taddr = t_lane + owner * 128;
                tmem_ld_32x32(taddr, v);
                tmem_ld_32x32(taddr + 32, v + 32);
                // allowed queries for this key: inside T, and not before the key if causal
                const long long rem_k = g.T - (long long)blk * kBlk;
                int lo = (g.causal && blk == qb) ? key : 0;
                if (key >= rem_k) lo = kBlk;  // key beyond T
                if (lo != 0 || m_lim != kBlk) {  // the diagonal block, or a block across T
#pragma unroll
                    for (int i = 0; i < 64; ++i) v[i] = (i >= lo && i < m_lim) ? v[i] : -CUDART_INF_F;
                }
                float best = max_of_64(v);
                best = warp_max(best);
                if (lane == 0) tl->part[r][c][wq & 1] = best;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tl->tmem_empty[slot]));
            return true;
        };
        for (int level = 0; level < levels; ++level) {
            const int lists = level == 0 ? 1 : R;
            for (int x = 0; x < lists; ++x) {
                const int li = level == 0 ? kR : x;
                if (level > 0) {
                    if (!mbar_wait(smem_u32(&tl->jobs_ready[x]), jr_par[x], tl, P.ws, 302)) return;
                    jr_par[x] ^= 1;
                }
                const int n = tl->n_jobs[li];
                const unsigned s_end = stage_seq + ((unsigned)(n + 1) >> 1);
                if (level == 0) {
                    // every stage serves all rows; rows grp, grp + 2 are this group's
                    for (unsigned s = stage_seq; s < s_end; ++s) {
                        const int c = 2 * (int)(s - stage_seq) + tile;
                        for (int r = grp; r < R; r += 2)
                            if (!reduce(s, r, li, c, n)) return;
                    }
                } else {
                    // one chain per stage; this group's are the stages with (s / kMmaWarps) % 2 == grp
                    unsigned s = stage_seq;
                    while (s < s_end) {
                        if ((int)((s / kMmaWarps) & 1u) != grp) { s = (s | (kMmaWarps - 1)) + 1; continue; }
                        if (!reduce(s, x, li, 2 * (int)(s - stage_seq) + tile, n)) return;
                        ++s;
                    }
                }
                stage_seq = s_end;
                // this list is done for rows r0..r1: tell the controller
                if (lane == 0) {
                    const int r0 = level == 0 ? 0 : x, r1 = level == 0 ? R : x + 1;
                    for (int r = r0; r < r1; ++r) mbar_arrive(smem_u32(&tl->scores_done[r]));
                    mbar_arrive(smem_u32(&tl->jobs_ack[li]));  // done reading this list
                }
            }
        }
    }
}

// Controller ----------------------------------------------------------------------------------------
// kMulti: several k per group with the score memory; false compiles the plain single-pass
// controller (its ranking step is on every group's critical path, so it carries nothing extra).
template <bool kMulti>
__device__ void controller_role(const Params &P, Tail *tl, int lane) {
    const Geom &g = P.g;
    const unsigned lt = (1u << lane) - 1u;
    unsigned sd_par[kR] = {0, 0, 0, 0};
    unsigned ack_par[kR + 1] = {0, 0, 0, 0, 0};  // phase of the next acknowledgement of each list
    // this CTA's score memory for the rows of its current group (several k only)
    unsigned long long *const cache = kMulti ? P.cache + (size_t)blockIdx.x * kR * g.N_k : nullptr;
    for (;;) {
        int id = 0;
        if (lane == 0) id = (int)atomicAdd(&P.ws->work_counter, 1u);
        id = __shfl_sync(0xffffffffu, id, 0);
        const bool done = id >= P.n_groups || *(volatile int *)&tl->abort_flag;
        int b = 0, kvh = 0, qb = 0, h0 = 0, R = 0;
        if (!done) {
            const int per = g.n_qb * P.n_chunks;
            const int bkv = id / per, rem = id % per;
            b = bkv / g.G; kvh = bkv % g.G;
            qb = g.n_qb - 1 - rem / P.n_chunks;  // late (expensive) query blocks first
            const int chunk = rem % P.n_chunks;
            h0 = kvh * g.hpg + chunk * kR;
            R = min(kR, g.hpg - chunk * kR);
        }
        const int q_lim = last_valid_block(g, qb);
        const unsigned tag = (unsigned)id + 1u;  // marks this group's entries of the score memory (0 = never written)
        const int n_pass = (!kMulti || done) ? 1 : P.mk.n;
        for (int pass = 0; pass < n_pass; ++pass) {
            // the group's k: all its rows are the same query block
            const int kq = done ? g.k_top : (kMulti ? P.mk.k[pass] : row_k(g, qb));
            const int levels = row_levels(g, kq);
            // initial nodes: lane i holds node i (the same for every row of the group)
            int f0 = (int)(((long long)lane * g.N_k) / kq), l0 = (int)(((long long)(lane + 1) * g.N_k) / kq) - 1;
            const bool v0 = !done && lane < kq && f0 <= l0 && f0 <= q_lim;
            const int m0 = (f0 + l0) / 2;
            const bool vl1 = v0, vr1 = v0 && m0 + 1 <= l0 && m0 + 1 <= q_lim;
            // Which of the two candidates does some row still lack a score for? (Without a score
            // memory: all of them.) A block on the first level's list is scored for every row.
            unsigned miss_l = vl1 ? (1u << R) - 1u : 0u, miss_r = vr1 ? (1u << R) - 1u : 0u;  // bit r: row r lacks it
            float cl[kR], cr[kR];
            if (kMulti && !done) {
#pragma unroll
                for (int r = 0; r < kR; ++r) {
                    cl[r] = cr[r] = -CUDART_INF_F;
                    if (r >= R) continue;
                    if (vl1) {
                        const unsigned long long e = __ldcg(cache + (size_t)r * g.N_k + f0);
                        if ((unsigned)(e >> 32) == tag) { cl[r] = __uint_as_float((unsigned)e); miss_l &= ~(1u << r); }
                    }
                    if (vr1) {
                        const unsigned long long e = __ldcg(cache + (size_t)r * g.N_k + m0 + 1);
                        if ((unsigned)(e >> 32) == tag) { cr[r] = __uint_as_float((unsigned)e); miss_r &= ~(1u << r); }
                    }
                }
            }
            const bool fl1 = miss_l != 0u, fr1 = miss_r != 0u;  // goes on the list
            const unsigned bl = __ballot_sync(0xffffffffu, fl1), br = __ballot_sync(0xffffffffu, fr1);
            const int c_l1 = __popc(bl & lt) + __popc(br & lt), c_r1 = c_l1 + (fl1 ? 1 : 0);
            // the previous list and record have been read by everybody (passes at once the first time)
            if (!mbar_wait(smem_u32(&tl->jobs_ack[kR]), ack_par[kR] ^ 1, tl, P.ws, 402)) return;
            ack_par[kR] ^= 1;
            if (fl1) tl->jobs_blk[kR][c_l1] = f0;
            if (fr1) tl->jobs_blk[kR][c_r1] = m0 + 1;
            const int n1 = __popc(bl) + __popc(br);
            if (lane == 0) {
                tl->n_jobs[kR] = n1;
                tl->grp_id = done ? -1 : id; tl->grp_b = b; tl->grp_kvh = kvh; tl->grp_qb = qb; tl->grp_h0 = h0; tl->grp_R = R;
                tl->grp_levels = levels;
                tl->grp_new_q = pass == 0;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tl->jobs_ready[kR]));
            if (done) return;

            int nf[kR], nl[kR], my_c[kR], n_nodes[kR], rb[kR];
            float ns[kR], cs[kR];
            bool has_r[kR], need[kR];
            unsigned tiles = 0;  // (row, block) tiles that had no score yet
            unsigned rt[kR];     // the same, row by row
#pragma unroll
            for (int r = 0; r < kR; ++r) {
                rt[r] = 0;
                if (r < R) rt[r] = (unsigned)(__popc(__ballot_sync(0xffffffffu, (miss_l >> r) & 1u)) + __popc(__ballot_sync(0xffffffffu, (miss_r >> r) & 1u)));
                tiles += rt[r];
            }
            for (int level = 0; level < levels; ++level) {
#pragma unroll
                for (int r = 0; r < kR; ++r) {
                    if (r >= R) continue;
                    if (!mbar_wait(smem_u32(&tl->scores_done[r]), sd_par[r], tl, P.ws, 401)) return;
                    sd_par[r] ^= 1;
                    // candidates of this lane's node: left (f : m) and right (m + 1 : l)
                    int f, l, m;
                    bool vl, vr;
                    float sl = -CUDART_INF_F, sr = -CUDART_INF_F;
                    if (level == 0) {
                        f = f0; l = l0; m = m0; vl = vl1; vr = vr1;
                        if (vl) sl = fl1 ? fmaxf(tl->part[r][c_l1][0], tl->part[r][c_l1][1]) : cl[r];
                        if (vr) sr = fr1 ? fmaxf(tl->part[r][c_r1][0], tl->part[r][c_r1][1]) : cr[r];
                        if (kMulti) {
                            if (fl1) __stcg(cache + (size_t)r * g.N_k + f0, cache_pack(tag, sl));
                            if (fr1) __stcg(cache + (size_t)r * g.N_k + m0 + 1, cache_pack(tag, sr));
                        }
                    } else {
                        f = nf[r]; l = nl[r]; m = (f + l) / 2;
                        vl = lane < n_nodes[r]; vr = has_r[r];
                        sl = ns[r];
                        if (vr) sr = need[r] ? fmaxf(tl->part[r][my_c[r]][0], tl->part[r][my_c[r]][1]) : cs[r];
                        if (kMulti && need[r]) __stcg(cache + (size_t)r * g.N_k + rb[r], cache_pack(tag, sr));
                    }
                    const Keep kp = select_topk(vl, sl, vr, sr, kq, lane);
                    const unsigned kl = __ballot_sync(0xffffffffu, kp.l), kr = __ballot_sync(0xffffffffu, kp.r);
                    const int pos_l = __popc(kl & lt) + __popc(kr & lt), pos_r = pos_l + (kp.l ? 1 : 0);
                    __syncwarp();
                    if (kp.l) { tl->node_f[pos_l] = f; tl->node_l[pos_l] = m; tl->node_s[pos_l] = sl; }
                    if (kp.r) { tl->node_f[pos_r] = m + 1; tl->node_l[pos_r] = l; tl->node_s[pos_r] = sr; }
                    __syncwarp();
                    n_nodes[r] = __popc(kl) + __popc(kr);
                    const bool live = lane < n_nodes[r];
                    nf[r] = live ? tl->node_f[lane] : 0;
                    nl[r] = live ? tl->node_l[lane] : -1;
                    ns[r] = live ? tl->node_s[lane] : -CUDART_INF_F;
                    if (level + 1 < levels) {
                        // next level: only right branches need a tile; left ones keep the node's score
                        const int mm = (nf[r] + nl[r]) / 2;
                        has_r[r] = live && nl[r] > nf[r] && mm + 1 <= q_lim;
                        rb[r] = mm + 1;
                        need[r] = has_r[r];
                        if (kMulti && has_r[r]) {  // an earlier pass (another k) may have scored it
                            const unsigned long long e = __ldcg(cache + (size_t)r * g.N_k + rb[r]);
                            if ((unsigned)(e >> 32) == tag) { cs[r] = __uint_as_float((unsigned)e); need[r] = false; }
                        }
                        const unsigned hb = __ballot_sync(0xffffffffu, need[r]);
                        my_c[r] = __popc(hb & lt);
                        if (!mbar_wait(smem_u32(&tl->jobs_ack[r]), ack_par[r] ^ 1, tl, P.ws, 403)) return;
                        ack_par[r] ^= 1;
                        if (need[r]) tl->jobs_blk[r][my_c[r]] = rb[r];
                        if (lane == 0) tl->n_jobs[r] = __popc(hb);
                        tiles += (unsigned)__popc(hb);
                        rt[r] += (unsigned)__popc(hb);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&tl->jobs_ready[r]));
                    } else {
                        // emit I[q, :]: first block of every surviving node, ascending, -1 padded
                        const long long o = (long long)pass * P.slab + (((long long)b * g.H + (h0 + r)) * g.n_qb + qb) * g.k_top;
                        if (lane < g.k_top) {
                            P.mask[o + lane] = live ? nf[r] : -1;
                            if (P.score != nullptr) P.score[o + lane] = live ? ns[r] : -CUDART_INF_F;
                        }
                        if (!kMulti && g.row_tiles != nullptr && lane == 0)
                            g.row_tiles[((long long)b * g.H + (h0 + r)) * g.n_qb + qb] = rt[r];
                    }
                }
            }
            if (lane == 0) {
                atomicAdd(&P.ws->tiles_scored, (unsigned long long)tiles);
                atomicAdd(&P.ws->rows, (unsigned long long)R);
            }
        }
    }
}

template <bool kMulti>
__global__ void __launch_bounds__(kThreads, 1)
mask_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k, Params P) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const unsigned q_smem = smem_u32(smem), k_smem = q_smem + kQBytes;
    Tail *tl = (Tail *)(smem + kQBytes + kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(smem_u32(&tl->full[i]), 1); mbar_init(smem_u32(&tl->empty[i]), 1); }
        for (int i = 0; i < kSlots; ++i) { mbar_init(smem_u32(&tl->tmem_full[i]), 1); mbar_init(smem_u32(&tl->tmem_empty[i]), 4); }
        mbar_init(smem_u32(&tl->q_full), 1);
        for (int i = 0; i <= kR; ++i) { mbar_init(smem_u32(&tl->jobs_ready[i]), 1); mbar_init(smem_u32(&tl->jobs_ack[i]), kListReaders); }
        for (int i = 0; i < kR; ++i) mbar_init(smem_u32(&tl->scores_done[i]), 4 * kEpiGroups);
        tl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {  // TMEM: all 512 columns (one CTA per SM)
        tmem_alloc_512(smem_u32(&tl->tmem_base));
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = tl->tmem_base;

    if (warp == 0 || warp == 14) {
        producer_role(P, &tmap_q, &tmap_k, tl, q_smem, k_smem, warp == 0 ? 0 : 1);
    } else if (warp == 1) {
        mma_role(P, tl, q_smem, k_smem, tmem_base, 0);
    } else if (warp == 2) {
        controller_role<kMulti>(P, tl, lane);
    } else if (warp == 3) {
        mma_role(P, tl, q_smem, k_smem, tmem_base, 1);
    } else if (warp == 12 || warp == 13) {
        mma_role(P, tl, q_smem, k_smem, tmem_base, warp - 10);
    } else if (warp >= 4 && warp < 12) {
        epilogue_role(P, tl, tmem_base, warp & 3, (warp - 4) >> 2, lane);
    }
    __syncwarp();

    // Teardown. After an abort, copies and MMAs may still be in flight: give every stage and slot
    // barrier a bounded chance to complete before shared memory and TMEM are given back.
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

// ----------------------------------------------------------------------------------------------
// Host side
// ----------------------------------------------------------------------------------------------
}  // namespace

bool mask_tc_supported(const Geom &g, int dtype) {
    return dtype == STREAM_BF16 && g.d == kD && g.bq == kBlk && g.bk == kBlk && g.k_top <= 32 && g.levels >= 1 &&
           tma_strides_ok(g);
}

namespace {
// CTAs of a launch and the groups they share.
stream_status launch_shape(const Geom &g, int *grid, long long *n_groups) {
    const int n_sm = sm_count();
    if (n_sm <= 0) { set_error("cannot read the SM count of the current device"); return STREAM_ERR_CUDA; }
    *n_groups = (long long)g.batch * g.G * g.n_qb * ((g.hpg + kR - 1) / kR);
    *grid = (int)(*n_groups < n_sm ? *n_groups : n_sm);
    return STREAM_OK;
}
}  // namespace

size_t mask_tc_score_memory_bytes(const Geom &g) {
    int grid = 0;
    long long n_groups = 0;
    if (launch_shape(g, &grid, &n_groups) != STREAM_OK) return 0;
    return (size_t)grid * kR * (size_t)g.N_k * sizeof(unsigned long long);
}

stream_status launch_mask_tc(const Geom &g, const void *q, const void *k, int32_t *mask, float *score,
                             WorkspaceHeader *ws, cudaStream_t st) {
    MultiK single = {};
    return launch_mask_tc_multi(g, single, q, k, mask, score, ws, nullptr, st);
}

stream_status launch_mask_tc_multi(const Geom &g, const MultiK &mk, const void *q, const void *k, int32_t *mask,
                                   float *score, WorkspaceHeader *ws, void *score_memory, cudaStream_t st) {
    if (((uintptr_t)q & 15) != 0 || ((uintptr_t)k & 15) != 0) {
        set_error("tensor-core mask kernel needs 16-byte aligned q and k");
        return STREAM_ERR_UNSUPPORTED;
    }
    CUtensorMap tq, tk;
    stream_status rc = make_map_bf16_d128(&tq, q, g.T, g.H, g.batch, g.qs_t, g.qs_h, g.qs_b, "q");
    if (rc != STREAM_OK) return rc;
    rc = make_map_bf16_d128(&tk, k, g.T, g.G, g.batch, g.ks_t, g.ks_h, g.ks_b, "k");
    if (rc != STREAM_OK) return rc;
    Params P;
    P.g = g;
    P.n_chunks = (g.hpg + kR - 1) / kR;
    long long n_groups = (long long)g.batch * g.G * g.n_qb * P.n_chunks;
    P.n_groups = (int)n_groups;
    P.mask = mask; P.score = score; P.ws = ws;
    P.mk = mk;
    P.cache = (unsigned long long *)score_memory;
    P.slab = (long long)g.batch * g.H * g.n_qb * g.k_top;
    int grid = 0;
    rc = launch_shape(g, &grid, &n_groups);
    if (rc != STREAM_OK) return rc;
    cudaError_t e = cudaSuccess;
    if (score_memory != nullptr) {  // tag 0 = "no score yet"
        e = cudaMemsetAsync(score_memory, 0, mask_tc_score_memory_bytes(g), st);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(score memory)");
    }
    if (mk.n >= 1 && score_memory == nullptr) { set_error("several k in one launch need the score memory"); return STREAM_ERR_WORKSPACE; }
    auto kern = mk.n >= 1 ? mask_tc_kernel<true> : mask_tc_kernel<false>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(mask_tc)");
    kern<<<grid, kThreads, kSmemBytes, st>>>(tq, tk, P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "mask_tc launch");
    return STREAM_OK;
}

}  // namespace stream
