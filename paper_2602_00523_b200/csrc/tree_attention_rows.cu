// Tree-masked verification attention over a paged bf16 KV cache (Section 2.2;
// Algorithm 1, the target pass over all tree tokens; Section 3.3 Phase 2), sm_100a:
// the streaming schedule for trees of more than 128 query rows per KV head.
// tree_attention.cu holds the form for smaller trees, the dispatch and the C entry points.
//
// Work decomposition.  The N tree nodes x G query heads that share one KV head form
// M = N*G query rows (<= 512).  An *item* is one (layer, sequence, KV head); its work
// is measured in steps of 128 keys (two 64-token pages).  All items are laid end to
// end and cut into equal ranges of steps, one range per *gang*; a gang is the 1 or 2
// CTAs (one per 256 query rows) that walk the same range side by side, so that the
// second CTA finds the K/V of the first in L2.  A kernel launch is one resident CTA
// per SM that loops over the segments of its range: whole items write their output
// directly, items cut by a range boundary leave unnormalised partial results that
// the merge kernel combines.  Nothing waits on another CTA.
//
// Inside a CTA (384 threads), per 128-key step and 128-row tile t:
//   TMA      : K and V tiles (2 pages x 2 d-halves) -> 128B-swizzled shared memory, rings of
//              3 K tiles and 2 V tiles, mbarriers; the two query tiles also arrive by TMA
//   tcgen05  : S_t = Q_t K^T (128 x 128, fp32) into TMEM; one warp issues for both row tiles, through
//              one elected lane, with warp-uniform descriptor arithmetic
//   softmax  : one warpgroup per row tile, one thread per row: tcgen05.ld S in four 32-column
//              chunks, online softmax in fp32 (log2 domain, lazy rescale), P -> bf16 back
//              into TMEM over the first 64 columns of S_t
//   tcgen05  : O_t += P_t V with P as the TMEM A operand, V MN-major from shared memory
// The two row tiles alternate on the tensor pipe: while one tile's warpgroup runs its softmax,
// the pipe works on the other tile.
// TMEM map (512 columns): S_t [128t, 128t+128), O_t [256+128t, 384+128t).
// All waits are bounded: on expiry the CTA records SAGE_STATUS_TIMEOUT, waits (bounded) for
// its copies and MMAs in flight, frees its TMEM and returns.
#include <cuda.h>

#include "sage_common.cuh"

namespace sage {
namespace rows {

constexpr int kRowTile = 128;                  // query rows per MMA tile
constexpr int kRowsPerCta = 2 * kRowTile;
constexpr int kStepKeys = 2 * kPageSize;       // keys per pipeline step
constexpr int kKStages = 3;                    // K tiles in flight
constexpr int kVStages = 2;                    // V tiles in flight
constexpr int kRing = 4;                       // barrier pairs of the copy ring (ring steps in flight <= 2)
constexpr int kPageHalfBytes = kPageSize * 64 * 2;          // one TMA box: 64 keys x 64-wide d-half = 8 KB
constexpr int kTileHalfBytes = kStepKeys * 64 * 2;          // one d-half of a 128-key tile: 16 KB
constexpr int kTileBytes = 2 * kTileHalfBytes;              // K or V tile of one step: 32 KB
constexpr int kQTileBytes = kRowTile * kHeadDim * 2;        // 32 KB
constexpr int kQHalfBytes = kRowTile * 64 * 2;              // one 64-wide d-half of a Q tile: 16 KB
constexpr int kAttnThreads = 384;              // 2 softmax warpgroups + one warpgroup of TMA warp, MMA warp and two idle warps
constexpr int kMinSteps = 2;                   // no range shorter than this (short contexts are latency-bound)

struct AttnParams {
    __nv_bfloat16* out;
    float* part_o;     // [gang][2][gang member][256 rows][128]   unnormalised
    float* part_ml;    // [gang][2][gang member][256 rows][2]     (reference max in log2 units, l)
    const int32_t* page_table;
    const int32_t* seq_len;
    const int32_t* parent;
    const int32_t* node_offsets;
    int32_t* status;
    int n_layers, batch, sum_nodes, n_pages, max_pages;
    int Hq, Hkv, G;
    int n_ctas, n_rp;          // CTAs of the launch; most CTAs a gang can have (row pairs of the largest possible tree)
    int select;                // which tree sizes this launch is for (schedule_selected)
    float scale_log2;          // sm_scale * log2(e)
    long long wait_cycles;     // budget of every on-device wait
    int producer_off;          // diagnostics: the TMA warp issues no copies (every consumer wait then runs out)
};

struct __align__(16) Shared {
    uint64_t kv_full[kRing];   // ring step r: the K tile of its step and the V tile of the step before have landed
    uint64_t kv_done[kRing];   // ring step r: every MMA that reads those tiles has finished
    uint64_t s_full[2];        // [row tile]: scores of a step are in TMEM
    uint64_t p_full[2];        // [row tile]: probabilities of a step are in TMEM
    uint64_t o_full[2];        // [row tile]: every MMA of the segment has finished
    uint64_t q_free;           // the segment's last score MMAs have read the query tiles
    uint64_t q_ready;          // the query tiles of the segment are in shared memory
    uint64_t drain;            // abort path: everything issued so far has retired
    long long range_begin, range_end;
    int first_lg, first_b, first_s0;
    int n_rp, n_gangs;         // CTAs per gang (row pairs of the largest tree of this batch) and gangs, found on the device
    uint32_t tmem_base;
    volatile int abort;
};
constexpr int kSmemBytes = 1024 /*align*/ + 2 * kQTileBytes + (kKStages + kVStages) * kTileBytes + (int)sizeof(Shared);
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA exceeded");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier ---------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Shared* sh, const AttnParams& p) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity)) return true;
        if (sh->abort) return false;
        if (clock64() - t0 > p.wait_cycles) {
            sh->abort = 1;
            report_status(p.status, SAGE_STATUS_TIMEOUT);
            return false;
        }
    }
}
// Used on the abort path only: gives up silently after the budget.
__device__ __forceinline__ void mbar_wait_quiet(uint64_t* bar, uint32_t parity, long long budget) {
    const long long t0 = clock64();
    while (!mbar_try(bar, parity) && clock64() - t0 < budget) {}
}

// ---- TMA ----------------------------------------------------------------------
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(smem_u32(bar)) : "memory");
}

// ---- tcgen05 --------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// One lane of a converged warp; the same lane every time for a full mask.
__device__ __forceinline__ bool elect_one() {
    uint32_t e;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(e));
    return e != 0;
}
// The helpers below are called by a whole converged warp so that their operands stay warp-uniform;
// only the `leader` lane executes the instruction.
__device__ __forceinline__ void tc_commit(bool leader, uint64_t* bar) {
    if (leader)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Shared-memory matrix descriptors are passed as (low word, high word): only the low word (start
// address and leading byte offset) varies between the MMAs of a kernel, so the issuing thread keeps
// 32-bit values and the 64-bit operand is assembled next to the instruction.
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "mov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (quadrant*32 + i)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte
// offsets in 16-byte units, version 1, 128-byte swizzle.  Low word: address and leading offset;
// high word: stride offset (1024 bytes between 8-row groups everywhere here), version, swizzle.
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
    return ((saddr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
}
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
// Instruction descriptor, kind::f16: D fp32, A and B bf16, M = 128, N as given.
constexpr uint32_t idesc_f16(uint32_t n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
constexpr uint32_t kIdescQK = idesc_f16(kStepKeys);              // S (128 x 128): A, B both K-major
constexpr uint32_t kIdescPV = idesc_f16(kHeadDim) | (1u << 16);  // O (128 x 128): B (= V) MN-major

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// ---- packed fp32 pairs (one instruction works on two values) ----
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// 2^x for a pair of x <= ~8 on the FMA and integer pipes instead of the special-function unit
// (which delivers only 16 results per clock per SM and would otherwise bound the softmax):
// x = n + f with n = round(x), f in [-0.5, 0.5]; 2^f by a cubic fitted to 7.5e-5 relative error
// (well below the 2^-9 rounding of the bf16 probabilities); n goes straight into the exponent bits.
// Inputs are clamped at -125, so that 2^x never leaves the normal range; -inf does not come here.
__device__ __forceinline__ void exp2_pair_fma(uint64_t x2, float& p0, float& p1) {
    constexpr float kMagic = 12582912.f;             // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
    float x0, x1;
    f2_unpack(x2, x0, x1);
    x2 = f2_pack(fmaxf(x0, -125.f), fmaxf(x1, -125.f));
    const uint64_t t2 = f2_add(x2, f2_pack(kMagic, kMagic));
    const uint64_t n2 = f2_add(t2, f2_pack(-kMagic, -kMagic));
    const uint64_t f2 = f2_fma(n2, f2_pack(-1.f, -1.f), x2);
    uint64_t q2 = f2_fma(f2, f2_pack(0.0551716685f, 0.0551716685f), f2_pack(0.2426111251f, 0.2426111251f));
    q2 = f2_fma(q2, f2, f2_pack(0.6932609677f, 0.6932609677f));
    q2 = f2_fma(q2, f2, f2_pack(0.9999280572f, 0.9999280572f));
    float t0, t1, q0, q1;
    f2_unpack(t2, t0, t1);
    f2_unpack(q2, q0, q1);
    p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
    p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}

#ifndef SAGE_EXP2_FMA_PAIRS
#define SAGE_EXP2_FMA_PAIRS 1       // of every 8 column pairs, evaluated on the FMA pipe instead of the SFU
#endif

// Maximum of 32 raw scores of one query row, folded into mx.
__device__ __forceinline__ void max_chunk(const uint32_t* sr, float& mx) {
    float m4[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float mq = max3(__uint_as_float(sr[q * 8]), __uint_as_float(sr[q * 8 + 1]), __uint_as_float(sr[q * 8 + 2]));
        mq = max3(mq, __uint_as_float(sr[q * 8 + 3]), __uint_as_float(sr[q * 8 + 4]));
        mq = max3(mq, __uint_as_float(sr[q * 8 + 5]), __uint_as_float(sr[q * 8 + 6]));
        m4[q] = fmaxf(mq, __uint_as_float(sr[q * 8 + 7]));
    }
    mx = fmaxf(max3(mx, m4[0], m4[1]), fmaxf(m4[2], m4[3]));
}

// 32 score columns of one query row: p = 2^(s * scale + neg_ref) packed to 16 bf16 pairs, and the
// fp32 sums of p in `acc`.  kEmu of every 8 column pairs take the FMA-pipe exp2.  Written in stages
// over the chunk so that neighbouring instructions are independent.
template <int kEmu>
__device__ __forceinline__ void exp_chunk(const uint32_t* sr, float scale, float neg_ref, uint32_t* pk,
                                          uint64_t (&acc)[2]) {
    const uint64_t scale2 = f2_pack(scale, scale), nref2 = f2_pack(neg_ref, neg_ref);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint64_t x2[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            x2[i] = f2_fma(f2_pack(__uint_as_float(sr[16 * h + 2 * i]), __uint_as_float(sr[16 * h + 2 * i + 1])), scale2, nref2);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float p0, p1;
            if (i < kEmu) {
                exp2_pair_fma(x2[i], p0, p1);
            } else {
                float x0, x1;
                f2_unpack(x2[i], x0, x1);
                p0 = fast_exp2(x0);
                p1 = fast_exp2(x1);
            }
            x2[i] = f2_pack(p0, p1);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i & 1] = f2_add(acc[i & 1], x2[i]);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float p0, p1;
            f2_unpack(x2[i], p0, p1);
            pk[8 * h + i] = pack_bf16(p0, p1);
        }
    }
}

// Scores of keys this row may not see become -inf: tree slot jt is visible iff it is an
// ancestor of (or is) the row's node; positions past the tree are never visible.
__device__ __forceinline__ void mask_chunk(uint32_t* sr, int pos0, int L, int N, uint64_t anc) {
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const int jt = pos0 + i - L;                      // tree slot; < 0 = prefix
        const bool vis = jt < 0 || (jt < N && ((anc >> jt) & 1ull));
        if (!vis) sr[i] = 0xff800000u;                    // -inf
    }
}

// The 128 scores of a step for one query row, TMEM -> registers: four loads, one wait.
__device__ __forceinline__ void load_scores(uint32_t s_taddr, uint32_t (&sr)[128]) {
    tmem_ld32(s_taddr, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
    tmem_ld32(s_taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
    tmem_ld32(s_taddr + 64, *reinterpret_cast<uint32_t(*)[32]>(&sr[64]));
    tmem_ld32(s_taddr + 96, *reinterpret_cast<uint32_t(*)[32]>(&sr[96]));
    tmem_wait_ld();
}

// O row *= alpha for the 32 rows of this warp (rare: only when a row maximum grew by more than 2^8).
__device__ __noinline__ void rescale_o_rows(uint32_t o_taddr, float alpha) {
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
        uint32_t orr[32];
        tmem_ld32(o_taddr + c * 32, orr);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
        tmem_st32(o_taddr + c * 32, orr);
    }
    tmem_wait_st();
}

// ---- schedule: items, ranges, segments ---------------------------------------------------
struct Item { int n0, N, L, steps, rp; };     // steps == 0: the sequence is skipped (and reported)

__device__ __forceinline__ Item load_item(const AttnParams& p, int b, int* err) {
    Item it;
    it.n0 = p.node_offsets[b];
    it.N = p.node_offsets[b + 1] - it.n0;
    it.L = p.seq_len[b];
    it.steps = 0;
    it.rp = 0;
    if (it.N < 1 || it.N > SAGE_MAX_NODES || it.n0 < 0 || it.n0 + it.N > p.sum_nodes) {
        *err = SAGE_STATUS_BAD_TREE;
        return it;
    }
    if (it.L < 0 || (long long)it.L + it.N > (long long)p.max_pages * kPageSize) {
        *err = SAGE_STATUS_BAD_PAGE;
        return it;
    }
    it.steps = (it.L + it.N + kStepKeys - 1) / kStepKeys;
    it.rp = (it.N * p.G + kRowsPerCta - 1) / kRowsPerCta;
    return it;
}

// Steps of all sequences of one (layer, KV head); called by a whole warp.
__device__ __forceinline__ int steps_per_head(const AttnParams& p, int lane, int* err) {
    int total = 0;
    for (int b0 = 0; b0 < p.batch; b0 += 32) {
        int s = 0;
        if (b0 + lane < p.batch) s = load_item(p, b0 + lane, err).steps;
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        total += s;
    }
    return total;
}
__device__ __forceinline__ int active_gangs(long long W, int n_gangs) {
    long long a = W / kMinSteps;
    if (a < 1) a = 1;
    return a < n_gangs ? (int)a : n_gangs;
}
__device__ __forceinline__ long long gang_begin(long long W, int n_act, int gang) { return (long long)gang * W / n_act; }
// Gang whose range holds position pos: the largest k with gang_begin(k) <= pos.
__device__ __forceinline__ int gang_of(long long W, int n_act, long long pos) {
    return (int)(((pos + 1) * n_act - 1) / W);
}
// Sequence b and step s0 inside it for offset `off` into one (layer, KV head); whole warp.
__device__ __forceinline__ void locate(const AttnParams& p, int lane, int off, int* b_out, int* s0_out) {
    int run = 0, err = 0;
    *b_out = p.batch;
    *s0_out = 0;
    for (int b0 = 0; b0 < p.batch; b0 += 32) {
        int s = 0;
        if (b0 + lane < p.batch) s = load_item(p, b0 + lane, &err).steps;
        int inc = s;
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        const unsigned hit = __ballot_sync(0xffffffffu, run + inc > off);
        if (hit) {
            const int l = __ffs(hit) - 1;
            const int incl = __shfl_sync(0xffffffffu, inc, l), sl = __shfl_sync(0xffffffffu, s, l);
            *b_out = b0 + l;
            *s0_out = off - (run + incl - sl);
            return;
        }
        run += __shfl_sync(0xffffffffu, inc, 31);
    }
}

struct Seg { int layer, g, b, n0, N, L, s0, s1, steps, rp; bool at_range_begin; };

// Walks the segments of a range; every thread that needs them runs its own copy.
struct SegIter {
    int remaining;      // steps of the range still to hand out
    int lg, b, s0;
    bool fresh;         // nothing handed out yet
    __device__ __forceinline__ void init(const Shared* sh) {
        remaining = (int)(sh->range_end - sh->range_begin);
        lg = sh->first_lg;
        b = sh->first_b;
        s0 = sh->first_s0;
        fresh = true;
    }
    __device__ __forceinline__ bool next(const AttnParams& p, Seg& sg) {
        int skipped = 0;
        while (remaining > 0 && b < p.batch && skipped <= p.batch) {
            int err = 0;
            const Item it = load_item(p, b, &err);
            if (it.steps == 0) {
                ++skipped;
                if (++b == p.batch) { b = 0; ++lg; }
                continue;
            }
            const int s1 = (it.steps - s0 <= remaining) ? it.steps : s0 + remaining;
            sg.layer = lg / p.Hkv; sg.g = lg % p.Hkv; sg.b = b;
            sg.n0 = it.n0; sg.N = it.N; sg.L = it.L;
            sg.s0 = s0; sg.s1 = s1; sg.steps = it.steps; sg.rp = it.rp;
            sg.at_range_begin = fresh;
            fresh = false;
            remaining -= s1 - s0;
            if (s1 == it.steps) {
                s0 = 0;
                if (++b == p.batch) { b = 0; ++lg; }
            } else {
                s0 = s1;
            }
            return true;
        }
        return false;
    }
};

__global__ void __launch_bounds__(kAttnThreads, 1)
tree_attention_rows_kernel(const AttnParams p, const __grid_constant__ CUtensorMap qmap,
                      const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128B swizzle pattern repeats every 1024 bytes of address
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                                 // [2 tiles][2 d-halves][128 rows][128 B]
    uint8_t* sK = sQ + 2 * kQTileBytes;                 // [kKStages][2 d-halves][128 keys][128 B]
    uint8_t* sV = sK + kKStages * kTileBytes;           // [kVStages][2 d-halves][128 keys][128 B]
    Shared* sh = reinterpret_cast<Shared*>(sV + kVStages * kTileBytes);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- the gangs of this launch and this gang's range of steps (warp 0 computes, everybody reads).
    // A gang has as many CTAs as the largest tree of the batch has row pairs, which only the device knows
    // when the caller's node arrays are larger than the trees in them.
    if (warp == 0) {
        int err = 0;
        const int rows_max = max_tree_rows(p.node_offsets, p.batch, p.sum_nodes, p.G, lane);
        const bool mine = schedule_selected(p.select, rows_max);
        const int n_rp = min(p.n_rp, max(1, (rows_max + kRowsPerCta - 1) / kRowsPerCta));
        const int n_gangs = p.n_ctas / n_rp;
        const int gang = blockIdx.x / n_rp;
        const int Wb = mine ? steps_per_head(p, lane, &err) : 0;
        if (err) report_status(p.status, err);
        const long long W = (long long)p.n_layers * p.Hkv * Wb;
        long long begin = 0, end = 0;
        int lg = 0, b = 0, s0 = 0;
        if (W > 0) {
            const int n_act = active_gangs(W, n_gangs);
            if (gang < n_act) {
                begin = gang_begin(W, n_act, gang);
                end = gang_begin(W, n_act, gang + 1);
            }
            if (end > begin) {
                lg = (int)(begin / Wb);
                locate(p, lane, (int)(begin % Wb), &b, &s0);
            }
        }
        if (lane == 0) {
            sh->range_begin = begin; sh->range_end = end;
            sh->first_lg = lg; sh->first_b = b; sh->first_s0 = s0;
            sh->n_rp = n_rp; sh->n_gangs = n_gangs;
        }
    }
    __syncthreads();
    if (sh->range_end <= sh->range_begin) return;       // uniform: nothing to do, nothing allocated yet
    const int n_rp = sh->n_rp;
    const int member = blockIdx.x % n_rp, gang = blockIdx.x / n_rp;

    // ---- set-up: barriers, TMEM
    if (tid == 0) {
        for (int i = 0; i < kRing; ++i) { mbar_init(&sh->kv_full[i], 1); mbar_init(&sh->kv_done[i], 1); }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&sh->s_full[t], 1);
            mbar_init(&sh->p_full[t], 4);               // one arrival per softmax warp
            mbar_init(&sh->o_full[t], 1);
        }
        mbar_init(&sh->q_free, 1);
        mbar_init(&sh->drain, 1);
        mbar_init(&sh->q_ready, 1);
        sh->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sh->tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;

    // Registers move from the copy / MMA warpgroup (which needs few) to the softmax warpgroups:
    // 4 warps give up 168 - 72 registers per thread, 8 warps take 216 - 168 each.
    if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 8) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            SegIter it;
            it.init(sh);
            Seg sg;
            // A segment of n steps takes n + 1 ring steps: ring step i carries the K tile of step s0 + i
            // (i < n) and the V tile of step s0 + i - 1 (i > 0), which is what the MMA warp consumes together
            // ([P V of the step before, scores of this step]); both land on one barrier.
            int rc = 0, kc = 0, vc = 0, nq = 0;          // ring steps, K tiles, V tiles, query loads issued so far
            bool ok = !p.producer_off;
            while (ok && it.next(p, sg)) {
                if (member >= sg.rp) continue;
                const int M = sg.N * p.G;
                const int n_rt = (M - member * kRowsPerCta > kRowTile) ? 2 : 1;
                const int32_t* pages = p.page_table + (size_t)sg.b * p.max_pages;
                const int n_pages_seq = (sg.L + sg.N + kPageSize - 1) / kPageSize;
                const int n = sg.s1 - sg.s0;
                int ids_prev[2] = {0, 0}, npg_prev = 0;
                for (int i = 0; i <= n; ++i) {
                    const int j = sg.s0 + i;
                    // page ids of step j (checked: they become TMA coordinates)
                    int ids[2] = {0, 0}, npg = 0;
                    if (i < n) {
                        npg = (2 * j + 1 < n_pages_seq) ? 2 : 1;
                        for (int pi = 0; pi < npg; ++pi) {
                            ids[pi] = pages[2 * j + pi];
                            if (ids[pi] < 0 || ids[pi] >= p.n_pages) {
                                report_status(p.status, SAGE_STATUS_BAD_PAGE);
                                ids[pi] = 0;
                            }
                        }
                    }
                    // the tiles that ring step rc - 2 used are free once its MMAs have finished
                    if (rc >= 2 && !mbar_wait(&sh->kv_done[(rc - 2) % kRing], ((rc - 2) / kRing) & 1, sh, p)) { ok = false; break; }
                    uint64_t* full = &sh->kv_full[rc % kRing];
                    mbar_expect_tx(full, (npg + (i > 0 ? npg_prev : 0)) * 2 * kPageHalfBytes);
                    if (i < n) {
                        const int kslot = kc % kKStages;
                        for (int pi = 0; pi < npg; ++pi)
                            for (int h = 0; h < 2; ++h)
                                tma_load_4d(smem_u32(sK + kslot * kTileBytes + h * kTileHalfBytes + pi * kPageHalfBytes), &kmap,
                                            h * 64, 0, ids[pi] * p.Hkv + sg.g, sg.layer, full);
                        ++kc;
                    }
                    if (i > 0) {
                        const int vslot = vc % kVStages;
                        for (int pi = 0; pi < npg_prev; ++pi)
                            for (int h = 0; h < 2; ++h)
                                tma_load_4d(smem_u32(sV + vslot * kTileBytes + h * kTileHalfBytes + pi * kPageHalfBytes), &vmap,
                                            h * 64, 0, ids_prev[pi] * p.Hkv + sg.g, sg.layer, full);
                        ++vc;
                    }
                    ++rc;
                    if (i == 0) {
                        // the segment's query tiles, once the previous segment's score MMAs have read theirs
                        if (nq > 0 && !mbar_wait(&sh->q_free, (nq - 1) & 1, sh, p)) { ok = false; break; }
                        mbar_expect_tx(&sh->q_ready, n_rt * kQTileBytes);
                        for (int t = 0; t < n_rt; ++t)
                            for (int h = 0; h < 2; ++h)
                                tma_load_5d(smem_u32(sQ + t * kQTileBytes + h * kQHalfBytes), &qmap, h * 64, 0, sg.g,
                                            sg.n0 + (member * kRowsPerCta + t * kRowTile) / p.G, sg.layer, &sh->q_ready);
                        ++nq;
                    }
                    ids_prev[0] = ids[0]; ids_prev[1] = ids[1]; npg_prev = npg;
                }
            }
            if (sh->abort) {
                // drain: every issued copy must land before the CTA may exit
                for (int n = max(0, rc - 2); n < rc; ++n)
                    mbar_wait_quiet(&sh->kv_full[n % kRing], (n / kRing) & 1, p.wait_cycles);
                if (nq > 0) mbar_wait_quiet(&sh->q_ready, (nq - 1) & 1, p.wait_cycles);
            }
        }
    } else if (warp == 9) {
        // =========================== MMA issuer ===========================
        // One thread issues for both row tiles, in blocks [P V of step j-1, scores of step j] per tile:
        // a tile's block runs on the tensor pipe while the other tile's warpgroup is in its softmax, and
        // the blocks of the two tiles never interleave (two issuers would finish both tiles' scores at
        // the same moment and leave the pipe idle during both softmaxes).  The whole instruction stream
        // sits in one single-thread region: a predicated branch around every MMA costs more issue time
        // than the MMA takes to execute.
        if (lane == 0) {
            // descriptors differ only in their 14-bit start-address field (bytes >> 4); shared memory ends below 256 KB
            const uint32_t dq = desc_lo(smem_u32(sQ), 16);
            const uint32_t dk = desc_lo(smem_u32(sK), 16);
            const uint32_t dv = desc_lo(smem_u32(sV), kTileHalfBytes);
            auto issue_qk = [&](int t, int slot) {
                // S_t = Q_t K^T: 8 slices of K = 16 over d = 128 (4 per 64-wide half)
                const uint32_t dqt = dq + ((t * kQTileBytes) >> 4);
                const uint32_t dks = dk + ((slot * kTileBytes) >> 4);
                const uint32_t s_tmem = tmem + t * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ss(s_tmem, dqt + (((ks >> 2) * kQHalfBytes + (ks & 3) * 32) >> 4),
                           dks + (((ks >> 2) * kTileHalfBytes + (ks & 3) * 32) >> 4), kDescHi, kIdescQK, ks > 0 ? 1u : 0u);
            };
            auto issue_pv = [&](int t, int slot, bool first) {
                // O_t += P_t V: 8 slices of K = 16 keys; P in TMEM (8 columns per slice), V MN-major
                const uint32_t dvs = dv + ((slot * kTileBytes) >> 4);
                const uint32_t s_tmem = tmem + t * 128, o_tmem = tmem + 256 + t * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts(o_tmem, s_tmem + ks * 8, dvs + ((ks * 2048) >> 4), kDescHi, kIdescPV, (first && ks == 0) ? 0u : 1u);
            };
            SegIter it;
            it.init(sh);
            Seg sg;
            int rc = 0, kc = 0, vc = 0, nq = 0;             // ring steps, K tiles, V tiles consumed; segments started
            int np[2] = {0, 0};                             // steps of each row tile whose probabilities were consumed
            bool ok = true;
            // Every synchronisation instruction costs this thread a couple of hundred clocks, during which
            // at most a few queued MMAs keep the pipe busy: the loop holds as few of them as the protocol
            // allows (one wait and one commit per ring step for the tiles, one of each per row tile).
            while (ok && it.next(p, sg)) {
                if (member >= sg.rp) continue;
                const int n_rt = (sg.N * p.G - member * kRowsPerCta > kRowTile) ? 2 : 1;
                const int s0 = sg.s0, s1 = sg.s1;
                ok = mbar_wait(&sh->q_ready, nq & 1, sh, p);
                ++nq;
                // ring step: the P V products of step j - 1 (when j > s0) and the scores of step j (when j < s1)
                for (int j = s0; ok && j <= s1; ++j) {
                    ok = mbar_wait(&sh->kv_full[rc % kRing], (rc / kRing) & 1, sh, p);
                    if (!ok) break;
                    const int kslot = kc % kKStages, vslot = vc % kVStages;
                    if (j < s1) ++kc;
                    if (j > s0) ++vc;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (t < n_rt) {
                            if (j > s0) {
                                // (the warpgroup zeroed the V rows past the end of the sequence before it arrived)
                                ok = mbar_wait(&sh->p_full[t], np[t] & 1, sh, p);
                                if (!ok) break;
                                ++np[t];
                                tc_fence_after();
                                issue_pv(t, vslot, j - 1 == s0);
                                if (j == s1) tc_commit(true, &sh->o_full[t]);   // every MMA of this tile's segment has been issued
                            }
                            if (j < s1) {
                                issue_qk(t, kslot);
                                tc_commit(true, &sh->s_full[t]);
                            }
                        }
                    }
                    if (!ok) break;
                    tc_commit(true, &sh->kv_done[rc % kRing]);
                    ++rc;
                    if (j == s1 - 1) tc_commit(true, &sh->q_free);          // the segment's last score MMAs read the query tiles
                }
            }
            if (!ok) {
                // abort: everything this thread has issued must retire before the TMEM and the tiles go away
                tc_commit(true, &sh->drain);
                mbar_wait_quiet(&sh->drain, 0, p.wait_cycles);
            }
        }
        __syncwarp();
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // =========================== softmax warpgroups ===========================
        const int t = warp >> 2;                        // row tile of this warpgroup
        const int r = tid & 127;                        // row inside the tile == TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_taddr = tmem + lane_base + t * 128;
        const uint32_t o_taddr = tmem + lane_base + 256 + t * 128;
        SegIter it;
        it.init(sh);
        Seg sg;
        int nsteps = 0, nseg = 0;                       // steps / segments this row tile has been through
        int rc0 = 0, vc0 = 0;                           // ring steps / V tiles of the CTA before the current segment
        bool ok = true;
        while (ok && it.next(p, sg)) {
            if (member >= sg.rp) continue;
            const int M = sg.N * p.G;
            const int rc_seg = rc0, vc_seg = vc0;       // this segment's first ring step / V tile
            rc0 += sg.s1 - sg.s0 + 1;
            vc0 += sg.s1 - sg.s0;
            if (t == 1 && M - member * kRowsPerCta <= kRowTile) continue;
            const int R = member * kRowsPerCta + t * kRowTile + r;
            const bool row_ok = R < M;
            const int node = row_ok ? R / p.G : 0;
            const bool warp_live = member * kRowsPerCta + t * kRowTile + (warp & 3) * 32 < M;
            uint64_t anc = 0;
            if (sg.s1 * kStepKeys > sg.L && row_ok) {
                // the segment reaches the tree part: this row's ancestor bitset (the G rows of a node
                // walk the same parent chain, at most N - 1 cached loads deep)
                bool bad = false;
                anc = ancestor_bits(p.parent + sg.n0, sg.N, node, &bad);
                if (bad) { report_status(p.status, SAGE_STATUS_BAD_TREE); anc = 1ull << node; }
            }
            float m_ref = -INFINITY, l_sum = 0.f;
            for (int j = sg.s0; j < sg.s1; ++j) {
                ok = mbar_wait(&sh->s_full[t], nsteps & 1, sh, p);
                if (!ok) break;
                const int valid = sg.L + sg.N - j * kStepKeys;      // keys of this step that exist
                if (valid < kStepKeys) {
                    // V rows past the end of the sequence may hold anything (a missing second page was not even
                    // copied): zero them so that 0 * V stays 0.  Each warp of the warpgroup takes a quarter of
                    // the rows (both warpgroups write the same zeros); the writes are ordered before this
                    // warp's arrival, which the P V product waits for.  The V tile of step j lands with ring
                    // step j - s0 + 1 of the segment.
                    const int rcv = rc_seg + (j - sg.s0) + 1;
                    ok = mbar_wait(&sh->kv_full[rcv % kRing], (rcv / kRing) & 1, sh, p);
                    if (!ok) break;
                    uint8_t* vb = sV + ((vc_seg + (j - sg.s0)) % kVStages) * kTileBytes;
                    for (int c = (warp & 3) * 32 + lane; c < (kStepKeys - valid) * 16; c += 128) {
                        const int vr = valid + c / 16, ch = c % 16;
                        *reinterpret_cast<uint4*>(vb + (ch >> 3) * kTileHalfBytes + vr * 128 + ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
                if (!warp_live) {
                    // none of this warp's 32 rows exists (ragged last tile): keep the barrier protocol
                    // going, leave the probabilities of these rows as they are; their outputs are never stored
                    ++nsteps;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh->p_full[t]);
                    continue;
                }
                tc_fence_after();
                const int pos0 = j * kStepKeys;
                const bool masked = pos0 + kStepKeys > sg.L;     // reaches into the tree part (or past the end)
                uint32_t sr[128];
                load_scores(s_taddr, sr);
                if (masked) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) mask_chunk(sr + 32 * c, pos0 + 32 * c, sg.L, sg.N, anc);
                }
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c) max_chunk(sr + 32 * c, mx);
                // lazy rescale: the reference moves only when the row max grew by more than 2^8 over it
                const float m_cand = mx * p.scale_log2;
                const bool grow = m_cand > m_ref + 8.0f;
                float alpha = 1.0f;
                if (grow) {
                    alpha = fast_exp2(m_ref - m_cand);              // 0 when m_ref was -inf
                    m_ref = m_cand;
                }
                // O_t *= alpha.  The P V product of the step before has finished: the scores of this step were
                // issued after it, and their completion is what this warp waited for above.
                if (j > sg.s0 && __any_sync(0xffffffffu, grow)) rescale_o_rows(o_taddr, alpha);
                const float neg_ref = (m_ref == -INFINITY) ? 0.f : -m_ref;
                // probabilities, packed to bf16 in place: chunk c (32 scores) leaves its 16 words at sr[16c ..]
                uint64_t acc[2] = {0ull, 0ull};
                if (masked) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) exp_chunk<0>(sr + 32 * c, p.scale_log2, neg_ref, sr + 16 * c, acc);   // may hold -inf
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) exp_chunk<SAGE_EXP2_FMA_PAIRS>(sr + 32 * c, p.scale_log2, neg_ref, sr + 16 * c, acc);
                }
                float sum_a, sum_b;
                f2_unpack(f2_add(acc[0], acc[1]), sum_a, sum_b);
                l_sum = l_sum * alpha + (sum_a + sum_b);
                uint32_t* pk = sr;
                tmem_st32(s_taddr, pk);                 // P over the first 64 columns of S_t
                tmem_st32(s_taddr + 32, pk + 32);
                tmem_wait_st();
                tc_fence_before();
                ++nsteps;
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh->p_full[t]);
            }
            if (!ok) break;
            // ---- epilogue: O_t / l -> bf16 output, or unnormalised partials for the merge
            ok = mbar_wait(&sh->o_full[t], nseg & 1, sh, p);
            ++nseg;
            if (!ok) break;
            tc_fence_after();
            const bool whole = (sg.s0 == 0 && sg.s1 == sg.steps);
            const float inv = (l_sum > 0.f) ? 1.0f / l_sum : 0.f;
            float* po = nullptr;
            __nv_bfloat16* oo = nullptr;
            if (whole) {
                const size_t row = (size_t)(sg.n0 + node) * p.Hq + sg.g * p.G + (row_ok ? R % p.G : 0);
                oo = p.out + ((size_t)sg.layer * p.sum_nodes * p.Hq + row) * kHeadDim;
            } else {
                const size_t pr = (((size_t)gang * 2 + (sg.at_range_begin ? 0 : 1)) * n_rp + member) * kRowsPerCta +
                                  t * kRowTile + r;
                po = p.part_o + pr * kHeadDim;
                if (row_ok) { p.part_ml[pr * 2] = m_ref; p.part_ml[pr * 2 + 1] = l_sum; }
            }
            if (warp_live) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t orr[32];
                    tmem_ld32(o_taddr + c * 32, orr);
                    tmem_wait_ld();
                    if (row_ok) {
                        if (oo) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                uint4 v;
                                v.x = pack_bf16(__uint_as_float(orr[8 * i + 0]) * inv, __uint_as_float(orr[8 * i + 1]) * inv);
                                v.y = pack_bf16(__uint_as_float(orr[8 * i + 2]) * inv, __uint_as_float(orr[8 * i + 3]) * inv);
                                v.z = pack_bf16(__uint_as_float(orr[8 * i + 4]) * inv, __uint_as_float(orr[8 * i + 5]) * inv);
                                v.w = pack_bf16(__uint_as_float(orr[8 * i + 6]) * inv, __uint_as_float(orr[8 * i + 7]) * inv);
                                *reinterpret_cast<uint4*>(oo + c * 32 + i * 8) = v;
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                *reinterpret_cast<uint4*>(po + c * 32 + i * 4) =
                                    make_uint4(orr[4 * i], orr[4 * i + 1], orr[4 * i + 2], orr[4 * i + 3]);
                        }
                    }
                }
            }
            tc_fence_before();                          // the next segment's first P V overwrites O_t
        }
    }
    // ---- teardown: every role is past its last TMEM access
    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// Merge of the items that a range boundary cut into segments.  Only a boundary between two gangs'
// ranges can cut an item, so the grid is (x = boundary, y = 32-row chunk): the block finds the item
// its boundary falls into, leaves if the boundary coincides with the item's start or if an earlier
// boundary already lies inside the same item (that block does the work), and otherwise combines the
// item's segments: which gangs hold them, and in which of their two partial slots, follows from
// the positions alone.
__global__ void __launch_bounds__(256) attention_rows_merge_kernel(AttnParams p) {
    __shared__ int s_Wb, s_b, s_s0, s_n_rp;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_cut = blockIdx.x + 1;                   // boundary between gang k_cut - 1 and gang k_cut
    if (warp == 0) {
        int err = 0, b = 0, s0 = 0;
        // the same gang layout as the attention kernel worked out
        const int rows_max = max_tree_rows(p.node_offsets, p.batch, p.sum_nodes, p.G, lane);
        const bool mine = schedule_selected(p.select, rows_max);
        const int n_rp = min(p.n_rp, max(1, (rows_max + kRowsPerCta - 1) / kRowsPerCta));
        const int Wb = mine ? steps_per_head(p, lane, &err) : 0;
        if (Wb > 0) {
            const long long W = (long long)p.n_layers * p.Hkv * Wb;
            const int n_act = active_gangs(W, p.n_ctas / n_rp);
            if (k_cut < n_act) locate(p, lane, (int)(gang_begin(W, n_act, k_cut) % Wb), &b, &s0);
        }
        if (lane == 0) { s_Wb = Wb; s_b = b; s_s0 = s0; s_n_rp = n_rp; }
    }
    __syncthreads();
    const int Wb = s_Wb;
    if (Wb <= 0) return;
    const int n_rp = s_n_rp;
    const long long W = (long long)p.n_layers * p.Hkv * Wb;
    const int n_act = active_gangs(W, p.n_ctas / n_rp);
    if (k_cut >= n_act || s_s0 == 0) return;            // no such boundary, or it falls between two items
    const long long cut = gang_begin(W, n_act, k_cut);
    const int lg = (int)(cut / Wb), b = s_b;
    int err = 0;
    const Item it = load_item(p, b, &err);
    const long long a = cut - s_s0;                     // position of the item's first step
    const int k_first = gang_of(W, n_act, a), k_last = gang_of(W, n_act, a + it.steps - 1);
    if (k_first != k_cut - 1) return;                   // an earlier boundary cuts the same item
    const bool first_mid_range = (a != gang_begin(W, n_act, k_first));
    const int M = it.N * p.G;
    const int layer = lg / p.Hkv, g = lg % p.Hkv;
    for (int i = 0; i < 4; ++i) {
        const int R = blockIdx.y * 32 + warp * 4 + i;
        if (R >= M) break;
        const int member = R / kRowsPerCta, Rl = R % kRowsPerCta;
        auto slot_row = [&](int k) -> size_t {
            const int slot = (k == k_first && first_mid_range) ? 1 : 0;
            return (((size_t)k * 2 + slot) * n_rp + member) * kRowsPerCta + Rl;
        };
        float mx = -INFINITY;
        for (int k = k_first + lane; k <= k_last; k += 32) {
            const size_t pr = slot_row(k);
            if (p.part_ml[pr * 2 + 1] > 0.f) mx = fmaxf(mx, p.part_ml[pr * 2]);
        }
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float lsum = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int k = k_first; k <= k_last; ++k) {
            const size_t pr = slot_row(k);
            const float l = p.part_ml[pr * 2 + 1];
            if (!(l > 0.f)) continue;
            const float w = exp2f(p.part_ml[pr * 2] - mx);
            lsum = fmaf(l, w, lsum);
            const float4 v = reinterpret_cast<const float4*>(p.part_o + pr * kHeadDim)[lane];
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
        }
        const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
        uint2 packed;
        packed.x = pack_bf16(acc.x * inv, acc.y * inv);
        packed.y = pack_bf16(acc.z * inv, acc.w * inv);
        const size_t row = (size_t)(it.n0 + R / p.G) * p.Hq + g * p.G + R % p.G;
        reinterpret_cast<uint2*>(p.out + ((size_t)layer * p.sum_nodes * p.Hq + row) * kHeadDim)[lane] = packed;
    }
}

// ---- host side ------------------------------------------------------------------------------
static int row_pairs(int sum_nodes, int G) {
    const int n = sum_nodes < SAGE_MAX_NODES ? sum_nodes : SAGE_MAX_NODES;      // a tree has at most that many nodes
    return (n * G + kRowsPerCta - 1) / kRowsPerCta;
}

// Two partial slots (head and tail of its range) per resident CTA, independent of the problem size.
size_t workspace_size(int n_ctas) { return (size_t)n_ctas * 2 * kRowsPerCta * (kHeadDim + 2) * sizeof(float); }

int launch(int n_ctas, int select, int n_layers, int n_pages, const int32_t* page_table, int max_pages_per_seq,
           const int32_t* seq_len, const int32_t* parent, const int32_t* node_offsets, int batch, int sum_nodes,
           int n_q_heads, int n_kv_heads, float sm_scale, void* out, void* ws, int32_t* status, long long wait_cycles,
           int producer_off, const CUtensorMap& qmap, const CUtensorMap& kmap, const CUtensorMap& vmap,
           cudaStream_t stream) {
    const int G = n_q_heads / n_kv_heads;
    AttnParams p{};
    p.n_rp = row_pairs(sum_nodes, G);
    p.n_ctas = (n_ctas / p.n_rp) * p.n_rp;          // whole gangs whatever the gang size turns out to be (1 or 2)
    p.select = select;
    p.out = (__nv_bfloat16*)out;
    p.part_o = (float*)ws;
    p.part_ml = (float*)ws + (size_t)n_ctas * 2 * kRowsPerCta * kHeadDim;
    p.page_table = page_table; p.seq_len = seq_len; p.parent = parent; p.node_offsets = node_offsets;
    p.status = status;
    p.n_layers = n_layers; p.batch = batch; p.sum_nodes = sum_nodes; p.n_pages = n_pages;
    p.max_pages = max_pages_per_seq; p.Hq = n_q_heads; p.Hkv = n_kv_heads; p.G = G;
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.wait_cycles = wait_cycles;
    p.producer_off = producer_off;
    // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SAGE_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(tree_attention_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) !=
            cudaSuccess)
            return SAGE_ERR_CUDA;
        attr_set[dev] = true;
    }
    tree_attention_rows_kernel<<<p.n_ctas, kAttnThreads, kSmemBytes, stream>>>(p, qmap, kmap, vmap);
    if (p.n_ctas > 1) {
        // one block per possible boundary between two gangs' ranges and 32-row chunk; those that find no cut item leave
        dim3 mg((unsigned)(p.n_ctas - 1), (unsigned)((p.n_rp * kRowsPerCta + 31) / 32));
        attention_rows_merge_kernel<<<mg, 256, 0, stream>>>(p);
    }
    return launch_status();
}

}  // namespace rows
}  // namespace sage
