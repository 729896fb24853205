// PTX wrappers and host helpers shared by the tcgen05 / TMA kernels of libstream (sm_100a only).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace stream {
namespace tc {

constexpr long long kWaitCycles = 1ll << 31;  // ~1 s: far beyond any legitimate wait

__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// The same, but the hardware may keep the thread suspended for up to `ns` nanoseconds while the
// phase is incomplete, instead of returning at once: far fewer shared-memory transactions than
// polling, and the shared-memory port is what these kernels run against.
__device__ __forceinline__ bool mbar_try_wait_suspend(unsigned bar, unsigned parity, unsigned ns) {
    unsigned ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}

// Non-blocking probe of an mbarrier phase.
__device__ __forceinline__ bool mbar_test_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait on an mbarrier phase. Returns false if the CTA is aborting, or if this wait ran
// out, in which case it raises the CTA's abort flag and records `code` (first one wins) with the
// block index in the two error words.
// (A kernel that moves registers between its warpgroups with setmaxnreg cannot call a separate
// function from the regions with different register counts: it defines STREAM_INLINE_SLOW_WAIT.)
#ifdef STREAM_INLINE_SLOW_WAIT
#define STREAM_SLOW_WAIT_ATTR __forceinline__
#else
#define STREAM_SLOW_WAIT_ATTR __noinline__
#endif
static __device__ STREAM_SLOW_WAIT_ATTR bool mbar_wait_slow(unsigned bar, unsigned parity, int *abort_flag, unsigned *err_code,
                                                   unsigned *err_info, unsigned code, long long limit) {
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait_suspend(bar, parity, 4000u)) return true;
        if (*(volatile int *)abort_flag) return false;
        if (clock64() - t0 > limit) {
            *(volatile int *)abort_flag = 1;
            if (atomicCAS(err_code, 0u, code) == 0u) *err_info = blockIdx.x;
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity, int *abort_flag, unsigned *err_code,
                                                  unsigned *err_info, unsigned code, long long limit = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;  // the common case costs one instruction
    return mbar_wait_slow(bar, parity, abort_flag, err_code, err_info, code, limit);
}

// True in exactly one lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
    unsigned pred;
    asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
    return pred != 0;
}

// mbar_wait_bounded for a whole converged warp: every lane waits, and all lanes get the same
// answer (false as soon as one lane saw the abort flag or ran out of time), so that the warp
// stays converged for the elect_one() that follows.
__device__ __forceinline__ bool mbar_wait_warp(unsigned bar, unsigned parity, int *abort_flag, unsigned *err_code,
                                               unsigned *err_info, unsigned code, long long limit = kWaitCycles) {
    const bool ok = mbar_wait_bounded(bar, parity, abort_flag, err_code, err_info, code, limit);
    return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void tma_load_4d(unsigned dst, const CUtensorMap *map, unsigned bar, int c0, int c1, int c2,
                                            int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"((unsigned long long)map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

__device__ __forceinline__ void tma_load_5d(unsigned dst, const CUtensorMap *map, unsigned bar, int c0, int c1, int c2,
                                            int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"((unsigned long long)map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Makes this thread's shared-memory writes visible to the async proxy (TMA, tcgen05.mma operands).
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// One tcgen05.mma (kind::f16, cta_group::1): D[tmem] (+)= A[smem] B[smem]. Both shared-memory
// descriptors are given as (low word, high word): the low word holds the start
// address in 16-byte units, so a K step is one 32-bit add on it; the high word never changes
// for a given operand layout.
__device__ __forceinline__ void tc_mma_bf16_split(unsigned d_tmem, unsigned a_lo, unsigned a_hi, unsigned b_lo,
                                                  unsigned b_hi, unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n.reg .pred p;\n.reg .b64 da, db;\nmov.b64 da, {%1, %2};\nmov.b64 db, {%3, %4};\nsetp.ne.b32 p, %6, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The same with an output-lane mask: bit i of the 128-bit vector {m0 (lanes 0..31), m1, m2, m3}
// set = accumulator lane i is left untouched by this instruction.
__device__ __forceinline__ void tc_mma_bf16_split_masked(unsigned d_tmem, unsigned a_lo, unsigned a_hi, unsigned b_lo,
                                                         unsigned b_hi, unsigned idesc, unsigned accumulate, unsigned m0,
                                                         unsigned m1, unsigned m2, unsigned m3) {
    asm volatile(
        "{\n.reg .pred p;\n.reg .b64 da, db;\nmov.b64 da, {%1, %2};\nmov.b64 db, {%3, %4};\nsetp.ne.b32 p, %6, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, {%7, %8, %9, %10}, p;\n}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(m0), "r"(m1), "r"(m2),
          "r"(m3)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc_512(unsigned smem_dst) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_512(unsigned tmem_base) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns of TMEM: thread i gets lane (base lane + i). Issue only;
// the registers are valid after tmem_ld_wait().
__device__ __forceinline__ void tmem_ld_32x32_issue(unsigned taddr, unsigned *r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
// Store 32 consecutive fp32 columns of this thread's TMEM lane (the inverse of the load above).
// Complete for later tcgen05 operations after tmem_st_wait().
__device__ __forceinline__ void tmem_st_32x32_issue(unsigned taddr, const unsigned *r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld_32x32(unsigned taddr, float *v) {
    unsigned r[32];
    tmem_ld_32x32_issue(taddr, r);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Maximum of three in one instruction.
__device__ __forceinline__ float max3(float a, float b, float c) {
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// Maximum of 64 values held in registers: four independent chains of three-input maxima instead of
// one chain of 64 (a quarter of the instructions' latency in a row, half the instructions).
__device__ __forceinline__ float max_of_64(const float *v) {
    float b0 = max3(v[0], v[1], v[2]), b1 = max3(v[3], v[4], v[5]), b2 = max3(v[6], v[7], v[8]), b3 = max3(v[9], v[10], v[11]);
#pragma unroll
    for (int i = 12; i < 60; i += 8) {
        b0 = max3(b0, v[i], v[i + 1]);
        b1 = max3(b1, v[i + 2], v[i + 3]);
        b2 = max3(b2, v[i + 4], v[i + 5]);
        b3 = max3(b3, v[i + 6], v[i + 7]);
    }
    b0 = max3(b0, v[60], v[61]);
    b1 = max3(b1, v[62], v[63]);
    return fmaxf(fmaxf(b0, b1), fmaxf(b2, b3));
}

__device__ __forceinline__ float warp_max(float x) {
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
    return r;
}

// Shared-memory matrix descriptor (sm_100 version 1) with 128-byte swizzle. Offsets in bytes.
//   K-major operand (rows of 128 bytes along K): sbo = distance between 8-row groups; lbo unused.
//   MN-major operand (rows of 128 bytes along M/N, one row per K index): sbo = distance between
//   8-K-index groups, lbo = distance between consecutive 64-element chunks along M/N.
// Bits: start address >> 4 in 0..13, lbo >> 4 in 16..29, sbo >> 4 in 32..45, version 1 in 46..47,
// swizzle mode 2 (128 bytes) in 61..63.
// Low and high words of that descriptor; (addr_bytes >> 4) is added to the low word per operand.
__device__ __forceinline__ unsigned desc_lo_sw128(unsigned addr, unsigned lbo) {
    return ((addr >> 4) & 0x3FFF) | (((lbo >> 4) & 0x3FFF) << 16);
}
__host__ __device__ constexpr unsigned desc_hi_sw128(unsigned sbo) { return ((sbo >> 4) & 0x3FFF) | (1u << 14) | (2u << 29); }

// kind::f16 instruction descriptor: D fp32, A and B bf16, A K-major, B K-major or MN-major.
__host__ __device__ constexpr unsigned idesc_bf16(unsigned M, unsigned N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

// Top-k of the (up to) 64 candidates a warp holds two per lane (a node's left and right branch):
// keep the k best by (score descending, candidate index ascending), the candidates numbered
// 2 * lane (left) and 2 * lane + 1 (right); k <= 32.
//
// The k-th largest score is found with a sorting network instead of counting ranks (4096
// comparisons, which made this the longest step of a row's level): the scores become unsigned
// keys of the same order (-0 first brought to +0, so that equal floats give equal keys; an absent
// candidate gets key 0, below every score), the 32 left keys are sorted descending and the 32
// right keys ascending across the lanes (one bitonic network, 15 exchange steps, both registers
// at once), the lane-wise maximum of the two is then the 32 largest keys as a bitonic sequence,
// five more steps sort it, and lane k - 1 holds the threshold. Every candidate above the threshold
// is kept; of those equal to it the first ones in candidate order, as many as are still missing.
struct Keep { bool l, r; };
__device__ __forceinline__ unsigned score_key(bool valid, float s) {
    const unsigned b = __float_as_uint(s + 0.f);
    return valid ? (b ^ ((b & 0x80000000u) ? 0xffffffffu : 0x80000000u)) : 0u;
}
__device__ __forceinline__ Keep select_topk(bool vl, float sl, bool vr, float sr, int k, int lane) {
    const int total = __popc(__ballot_sync(0xffffffffu, vl)) + __popc(__ballot_sync(0xffffffffu, vr));
    if (total <= k) return {vl, vr};
    const unsigned kl = score_key(vl, sl), kr = score_key(vr, sr);
    unsigned a = kl, b = kr;  // a: sorted descending over the lanes, b: ascending
#pragma unroll
    for (int k2 = 2; k2 <= 32; k2 <<= 1) {
#pragma unroll
        for (int j = k2 >> 1; j > 0; j >>= 1) {
            const unsigned oa = __shfl_xor_sync(0xffffffffu, a, j), ob = __shfl_xor_sync(0xffffffffu, b, j);
            // in an ascending network the lower lane of a pair takes the minimum inside an "up" block
            const bool first = (((lane & j) == 0) == ((lane & k2) == 0));
            a = first ? max(a, oa) : min(a, oa);
            b = first ? min(b, ob) : max(b, ob);
        }
    }
    unsigned c = max(a, b);  // the 32 largest of the 64 keys, a bitonic sequence over the lanes
#pragma unroll
    for (int j = 16; j > 0; j >>= 1) {
        const unsigned oc = __shfl_xor_sync(0xffffffffu, c, j);
        c = ((lane & j) == 0) ? max(c, oc) : min(c, oc);
    }
    const unsigned thr = __shfl_sync(0xffffffffu, c, k - 1);  // the k-th largest key (with multiplicity)
    const bool gl = kl > thr, gr = kr > thr, el = kl == thr, er = kr == thr;
    const int missing = k - __popc(__ballot_sync(0xffffffffu, gl)) - __popc(__ballot_sync(0xffffffffu, gr));
    const unsigned bel = __ballot_sync(0xffffffffu, el), ber = __ballot_sync(0xffffffffu, er);
    const unsigned lt = (1u << lane) - 1u;
    const int pos_l = __popc(bel & lt) + __popc(ber & lt), pos_r = pos_l + (el ? 1 : 0);
    return {vl && (gl || (el && pos_l < missing)), vr && (gr || (er && pos_r < missing))};
}

struct Ring {  // position in a ring of barriers with phase tracking
    int idx = 0;
    unsigned phase = 0;
    __device__ void advance(int n) {
        if (++idx == n) { idx = 0; phase ^= 1; }
    }
};

// ----------------------------------------------------------------------------------------------
// Host side
// ----------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// [batch, heads, T, 128] bf16 with element strides -> 4-D map with a box of 64 channels x box_rows
// tokens (64 unless told otherwise), 128-byte swizzle. Rows beyond T read as zeros.
inline stream_status make_map_bf16_d128(CUtensorMap *map, const void *base, long long T, int heads, int batch,
                                        long long s_t, long long s_h, long long s_b, const char *what, int box_rows = 64) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return STREAM_ERR_CUDA; }
    // extents of 1 may come with arbitrary strides: give them a well-formed one
    if (heads == 1) s_h = s_t * T;
    if (batch == 1) s_b = s_h * heads;
    cuuint64_t dims[4] = {128, (cuuint64_t)T, (cuuint64_t)heads, (cuuint64_t)batch};
    cuuint64_t strides[3] = {(cuuint64_t)s_t * 2, (cuuint64_t)s_h * 2, (cuuint64_t)s_b * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1}, estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled(%s) failed with %d", what, (int)r); return STREAM_ERR_CUDA; }
    return STREAM_OK;
}

// The same tensor seen as [batch, heads, 2 channel halves, T, 64]: one box brings a whole
// 64-token x 128-channel tile (16 KB) as [half][64 rows][128 B], the layout of a 128-byte-swizzled
// K-major (or, read along the rows, MN-major) tcgen05 operand. With heads_in_box = 2 the two
// heads h, h + 1 land as [half][head][64 rows][128 B]: a 128-row operand per half.
// Coordinates: (0, token, head, 0, batch) with the half as dimension 3.
inline stream_status make_map5_bf16_d128(CUtensorMap *map, const void *base, long long T, int heads, int batch,
                                         long long s_t, long long s_h, long long s_b, int heads_in_box, const char *what) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return STREAM_ERR_CUDA; }
    if (heads == 1) s_h = s_t * T;
    if (batch == 1) s_b = s_h * heads;
    cuuint64_t dims[5] = {64, (cuuint64_t)T, (cuuint64_t)heads, 2, (cuuint64_t)batch};
    cuuint64_t strides[4] = {(cuuint64_t)s_t * 2, (cuuint64_t)s_h * 2, 128, (cuuint64_t)s_b * 2};
    cuuint32_t box[5] = {64, 64, (cuuint32_t)heads_in_box, 2, 1}, estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled(%s) failed with %d", what, (int)r); return STREAM_ERR_CUDA; }
    return STREAM_OK;
}

inline bool tma_strides_ok(const Geom &g) {
    auto ok = [](long long s) { return s % 8 == 0; };  // 16-byte multiples
    return ok(g.qs_t) && ok(g.qs_h) && ok(g.qs_b) && ok(g.ks_t) && ok(g.ks_h) && ok(g.ks_b);
}

inline int sm_count() {
    static int n_sm = 0;
    if (n_sm == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            n_sm = 0;
    }
    return n_sm;
}

}  // namespace tc
}  // namespace stream
