// Tree-masked verification attention over a paged bf16 KV cache (Section 2.2;
// Algorithm 1, the target pass over all tree tokens; Section 3.3 Phase 2), sm_100a:
// the C entry points, the choice of schedule, and the streaming kernel for trees of one
// row tile.  tree_attention_rows.cu holds the streaming kernel for two row tiles per CTA,
// tree_attention_split.cu the split schedule.
//
// Work decomposition.  The N tree nodes x G query heads that share one KV head form
// M = N*G query rows; here M <= 128, one row tile (the pair form takes more: see below).
// An *item* is one (layer, sequence, KV head); its work is measured in steps of 128 keys
// (two 64-token pages).  All items are laid end to end and cut into equal ranges of steps,
// one range per *gang* (one CTA; in the pair form the CTA pairs that cover a tree's row
// tiles).  A kernel launch is one resident CTA per SM that loops over the segments of its
// range: whole items write their output directly, items cut by a range boundary leave
// unnormalised partial results that attention_merge_kernel combines.  No CTA waits on
// another one outside its pair.
//
// Inside a CTA (384 threads): tensor memory holds two slots t of (S_t 128 x 128 fp32 scores,
// O_t 128 x 128 fp32 accumulator).  Both slots work for the same 128 query rows: slot t takes
// the steps s0 + t, s0 + t + 2, ... of a segment, so that the softmax of one step runs while
// the tensor pipe works on the next step (with one slot the chain scores -> softmax -> P V of
// a row tile is strictly serial); the two accumulators are combined in the epilogue.
//   TMA      : K and V tiles (2 pages x 2 d-halves) -> 128B-swizzled shared memory, rings of
//              3 K tiles and 3 V tiles, mbarriers; the query tile also arrives by TMA
//   tcgen05  : S_t = Q K^T into TMEM; one thread issues for both slots, in blocks
//              [P V of step i-2, scores of step i]
//   softmax  : one warpgroup per slot, one thread per row: tcgen05.ld S in four 32-column
//              chunks, online softmax in fp32 (log2 domain, lazy rescale), P -> bf16 back
//              into TMEM over the first 64 columns of S_t
//   tcgen05  : O_t += P_t V with P as the TMEM A operand, V MN-major from shared memory
// A 128 x 64 score MMA occupies the tensor pipe exactly as long as a 128 x 128 one (64 clocks
// per K=16 slice, measured), hence the 128-key step.
// TMEM map (512 columns): S_t [128t, 128t+128), O_t [256+128t, 384+128t).
//
// Pair form (tree_attention_kernel<true>, forced for measurements only): clusters of two CTAs
// with one MMA stream (cta_group::2, M = 256), one row tile per CTA; each CTA holds half of every
// K tile and half of every V tile, so a step's K and V enter the pair's shared memory once.
//
// All waits are bounded: on expiry the CTA (both CTAs of a pair) records SAGE_STATUS_TIMEOUT,
// waits (bounded) for its copies and MMAs in flight, frees its TMEM and returns.
#include <cuda.h>

#include <mutex>

#include "sage_common.cuh"

namespace sage {

constexpr int kRowTile = 128;                  // query rows per MMA tile
constexpr int kRowsPerCta = kRowTile;          // one row tile per CTA; its steps alternate between two slots
constexpr int kStepKeys = 2 * kPageSize;       // keys per pipeline step
constexpr int kPageHalfBytes = kPageSize * 64 * 2;          // one TMA box: 64 keys x 64-wide d-half = 8 KB
constexpr int kTileHalfBytes = kStepKeys * 64 * 2;          // one d-half of a 128-key tile: 16 KB
constexpr int kTileBytes = 2 * kTileHalfBytes;              // K or V tile of one step: 32 KB
constexpr int kMaxRing = 8;
// The kernel comes in two forms.  Single: one CTA holds the whole K and V tile of a step.  Pair: two
// CTAs of a cluster (the two SMs of a TPC) work on two row tiles with one MMA stream (cta_group::2, M = 256);
// each holds half of every K tile (64 of the 128 keys) and half of every V tile (64 of the 128 head
// dimensions), so a step's K and V enter the pair's shared memory once.
template <bool kPair>
struct Cfg {
    static constexpr int kStages = kPair ? 6 : 3;                       // K tiles, and V tiles, in flight per CTA
    static constexpr int kDepth = kStages;                              // ring steps the copies run ahead of the MMAs
    static constexpr int kRing = kStages + 1;                           // barrier pairs of the copy ring (> kDepth)
    static constexpr int kTile = kPair ? kTileBytes / 2 : kTileBytes;   // this CTA's part of a step's K (or V) tile
    static constexpr int kKHalf = kTile / 2;                            // distance between the two d-halves of its K part
    static_assert(kRing <= kMaxRing, "ring barriers");
};
constexpr int kQTileBytes = kRowTile * kHeadDim * 2;        // 32 KB
constexpr int kQHalfBytes = kRowTile * 64 * 2;              // one 64-wide d-half of a Q tile: 16 KB
constexpr int kAttnThreads = 384;              // 2 softmax warpgroups + one warpgroup of TMA warp, MMA warp and two idle warps
constexpr int kMinSteps = 2;                   // no range shorter than this (short contexts are latency-bound)
constexpr long long kWaitCyclesDefault = 4000000000ll;   // ~2 s at 2 GHz: far beyond any legitimate wait

struct AttnParams {
    __nv_bfloat16* out;
    float* part_o;     // [gang][2][gang member][128 rows][128]   unnormalised
    float* part_ml;    // [gang][2][gang member][128 rows][2]     (reference max in log2 units, l)
    const int32_t* page_table;
    const int32_t* seq_len;
    const int32_t* parent;
    const int32_t* node_offsets;
    int32_t* status;
    int n_layers, batch, sum_nodes, n_pages, max_pages;
    int Hq, Hkv, G;
    int n_gangs, n_rp;         // gangs in the launch, CTAs per gang (row tiles of the largest possible tree)
    float scale_log2;          // sm_scale * log2(e)
    long long wait_cycles;     // budget of every on-device wait
    int producer_off;          // diagnostics: the TMA warp issues no copies (every consumer wait then runs out)
    int select;                // which tree sizes this launch is for (schedule_selected)
};

struct __align__(16) Shared {
    uint64_t kv_full[kMaxRing];    // ring step r: the K tile of its step and the V tile of two steps back have landed
    uint64_t kv_done[kMaxRing];    // ring step r: every MMA that reads those tiles has finished
    uint64_t s_full[2];        // [slot]: scores of a step are in TMEM
    uint64_t p_full[2];        // [slot]: probabilities of a step are in TMEM
    uint64_t o_full[2];        // [slot]: every MMA of the slot's part of the segment has finished
    uint64_t epi_done;         // the softmax warps have read both accumulators of the segment
    uint64_t q_free;           // the segment's last score MMAs have read the query tile
    uint64_t q_ready;          // the query tile of the segment is in shared memory
    uint64_t drain;            // abort path: everything issued so far has retired
    volatile uint32_t eflag[2][4];     // [slot][quadrant]: segment number whose (reference, sum) this warp has posted
    long long range_begin, range_end;
    int first_lg, first_b, first_s0;
    uint32_t tmem_base;
    uint32_t peer_abort;       // pair form: cluster address of the other CTA's abort flag (0: none)
    volatile int abort;
};
// the same for both forms: a query tile and 6 x 32 KB (or 12 x 16 KB) of K and V
constexpr int kSmemBytes = 1024 /*align*/ + kQTileBytes + 6 * kTileBytes + (int)sizeof(Shared);
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA exceeded");
static_assert(2 * Cfg<false>::kStages * Cfg<false>::kTile == 6 * kTileBytes && 2 * Cfg<true>::kStages * Cfg<true>::kTile == 6 * kTileBytes, "ring size");

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
// kCluster: the barrier also takes arrivals from the other CTA of the pair
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    if (kCluster)
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_addr(const volatile void* ptr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(const_cast<const void*>(ptr))), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// The CTA (and, in the pair form, its partner) stops: every wait returns false from here on.
__device__ __forceinline__ void raise_abort(Shared* sh) {
    sh->abort = 1;
    if (sh->peer_abort) asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(sh->peer_abort), "r"(1) : "memory");
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Shared* sh, const AttnParams& p) {
    if (mbar_try<kCluster>(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try<kCluster>(bar, parity)) return true;
        if (sh->abort) return false;
        if (clock64() - t0 > p.wait_cycles) {
            raise_abort(sh);
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
// Issued by the one thread that issues the MMAs.
// Pair form: the arrival goes to the barrier at this offset in both CTAs, or (`both` false) in this one only.
template <bool kPair>
__device__ __forceinline__ void tc_commit_to(uint64_t* bar, bool both = true) {
    if (!kPair) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
    } else if (both) {
        const uint16_t mask = 3;
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(smem_u32(bar)), "h"(mask) : "memory");
    } else {
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
    }
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
// The same two for a CTA pair: M = 256, each CTA supplies its 128 rows of A and its half of B's N extent.
__device__ __forceinline__ void mma2_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma2_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "mov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc) : "memory");
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
__device__ __forceinline__ void tmem_st2(uint32_t taddr, uint32_t a, uint32_t b) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};" ::"r"(taddr), "r"(a), "r"(b) : "memory");
}
// two columns, waited for
__device__ __forceinline__ void tmem_ld2(uint32_t taddr, uint32_t& a, uint32_t& b) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];" : "=r"(a), "=r"(b) : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
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
constexpr uint32_t idesc_f16(uint32_t n, uint32_t m = 128u) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((m >> 4) << 24);
}
constexpr uint32_t kIdescQK = idesc_f16(kStepKeys);              // S (128 x 128): A, B both K-major
constexpr uint32_t kIdescPV = idesc_f16(kHeadDim) | (1u << 16);  // O (128 x 128): B (= V) MN-major
constexpr uint32_t kIdescQK2 = idesc_f16(kStepKeys, 256u);       // the same over the 256 rows of a CTA pair
constexpr uint32_t kIdescPV2 = idesc_f16(kHeadDim, 256u) | (1u << 16);

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

template <bool kPair>
__global__ void __launch_bounds__(kAttnThreads, 1)
tree_attention_kernel(const AttnParams p, const __grid_constant__ CUtensorMap qmap,
                      const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128B swizzle pattern repeats every 1024 bytes of address
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                                 // [2 d-halves][128 rows][128 B]
    using C = Cfg<kPair>;
    constexpr int kStages = C::kStages, kDepth = C::kDepth, kRing = C::kRing, kTile = C::kTile, kKHalf = C::kKHalf;
    // single: K [stage][2 d-halves][128 keys][128 B], V the same; pair: K [stage][2 d-halves][this CTA's 64 keys][128 B],
    // V [stage][128 keys][this CTA's 64-wide d-half = 128 B]
    uint8_t* sK = sQ + kQTileBytes;
    uint8_t* sV = sK + kStages * kTile;
    Shared* sh = reinterpret_cast<Shared*>(sV + kStages * kTile);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // member = row tile of the tree that this CTA owns; a pair is two consecutive members
    const int member = blockIdx.x % p.n_rp, gang = blockIdx.x / p.n_rp;
    const int crank = kPair ? (member & 1) : 0;                     // rank in the pair; rank 0 issues the MMAs
    const bool is_lead = crank == 0;
    const int member0 = kPair ? (member & ~1) : member;            // first member of the pair: decides whether an item is this pair's

    // ---- this gang's range of steps (warp 0 computes, everybody reads)
    if (warp == 0) {
        int err = 0;
        const bool mine = schedule_selected(p.select, max_tree_rows(p.node_offsets, p.batch, p.sum_nodes, p.G, lane));
        const int Wb = mine ? steps_per_head(p, lane, &err) : 0;
        if (err) report_status(p.status, err);
        const long long W = (long long)p.n_layers * p.Hkv * Wb;
        long long begin = 0, end = 0;
        int lg = 0, b = 0, s0 = 0;
        if (W > 0) {
            const int n_act = active_gangs(W, p.n_gangs);
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
        }
    }
    __syncthreads();
    if (sh->range_end <= sh->range_begin) return;       // uniform: nothing to do, nothing allocated yet

    // ---- set-up: barriers, TMEM
    if (tid == 0) {
        // Pair form: the leader's "landed" barriers also take the relayed arrival of the partner's copies, and
        // the barriers that the softmax warps arrive on count the warps of both CTAs.
        const int lands = (kPair && is_lead) ? 2 : 1;
        for (int i = 0; i < kRing; ++i) { mbar_init(&sh->kv_full[i], lands); mbar_init(&sh->kv_done[i], 1); }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&sh->s_full[t], 1);
            mbar_init(&sh->p_full[t], kPair ? 8 : 4);   // one arrival per softmax warp of the slot
            mbar_init(&sh->o_full[t], 1);
        }
        mbar_init(&sh->epi_done, kPair ? 16 : 8);       // one arrival per softmax warp
        mbar_init(&sh->q_free, 1);
        mbar_init(&sh->drain, 1);
        mbar_init(&sh->q_ready, lands);
        sh->abort = 0;
        sh->peer_abort = kPair ? cluster_addr(&sh->abort, crank ^ 1) : 0u;
        for (int i = 0; i < 8; ++i) (&sh->eflag[0][0])[i] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        if (kPair) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&sh->tmem_base)), "r"(512) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&sh->tmem_base)), "r"(512) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (kPair) {
        // both CTAs' barriers and tensor memory exist before either touches the other's
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    // where the softmax warps arrive: the leader's barriers
    const uint32_t lead_p_full[2] = {kPair ? cluster_addr(&sh->p_full[0], 0) : 0u, kPair ? cluster_addr(&sh->p_full[1], 0) : 0u};
    const uint32_t lead_epi_done = kPair ? cluster_addr(&sh->epi_done, 0) : 0u;

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
            // A segment of n steps takes n + 2 ring steps: ring step i carries the K tile of step s0 + i
            // (i < n) and the V tile of step s0 + i - 2 (i >= 2), which is what the MMA warp consumes together
            // ([P V of the step two back, scores of this step]); both land on one barrier.
            int rc = 0, kc = 0, vc = 0, nq = 0;          // ring steps, K tiles, V tiles, query loads issued so far
            bool ok = !p.producer_off;
            while (ok && it.next(p, sg)) {
                if (member0 >= sg.rp) continue;
                const int32_t* pages = p.page_table + (size_t)sg.b * p.max_pages;
                const int n_pages_seq = (sg.L + sg.N + kPageSize - 1) / kPageSize;
                const int n = sg.s1 - sg.s0;
                int ids_a[2] = {0, 0}, npg_a = 0;        // pages of step i - 1
                int ids_b[2] = {0, 0}, npg_b = 0;        // pages of step i - 2
                for (int i = 0; i < n + 2; ++i) {
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
                    // the tiles that ring step rc - kDepth used are free once its MMAs have finished
                    if (rc >= kDepth &&
                        !mbar_wait(&sh->kv_done[(rc - kDepth) % kRing], ((rc - kDepth) / kRing) & 1, sh, p)) { ok = false; break; }
                    uint64_t* full = &sh->kv_full[rc % kRing];
                    const int npv = i >= 2 ? npg_b : 0;
                    if (!kPair) {
                        mbar_expect_tx(full, (npg + npv) * 2 * kPageHalfBytes);
                        if (i < n) {
                            const int kslot = kc % kStages;
                            for (int pi = 0; pi < npg; ++pi)
                                for (int h = 0; h < 2; ++h)
                                    tma_load_4d(smem_u32(sK + kslot * kTile + h * kKHalf + pi * kPageHalfBytes), &kmap,
                                                h * 64, 0, ids[pi] * p.Hkv + sg.g, sg.layer, full);
                        }
                        for (int pi = 0; pi < npv; ++pi)
                            for (int h = 0; h < 2; ++h)
                                tma_load_4d(smem_u32(sV + (vc % kStages) * kTile + h * kTileHalfBytes + pi * kPageHalfBytes), &vmap,
                                            h * 64, 0, ids_b[pi] * p.Hkv + sg.g, sg.layer, full);
                    } else {
                        // this CTA's share: page `crank` of the K tile (both d-halves), d-half `crank` of the V tile (both pages)
                        const bool my_k = i < n && crank < npg;
                        mbar_expect_tx(full, ((my_k ? 2 : 0) + npv) * kPageHalfBytes);
                        if (my_k)
                            for (int h = 0; h < 2; ++h)
                                tma_load_4d(smem_u32(sK + (kc % kStages) * kTile + h * kKHalf), &kmap,
                                            h * 64, 0, ids[crank] * p.Hkv + sg.g, sg.layer, full);
                        for (int pi = 0; pi < npv; ++pi)
                            tma_load_4d(smem_u32(sV + (vc % kStages) * kTile + pi * kPageHalfBytes), &vmap,
                                        crank * 64, 0, ids_b[pi] * p.Hkv + sg.g, sg.layer, full);
                    }
                    if (i < n) ++kc;
                    if (i >= 2) ++vc;
                    ++rc;
                    if (i == 0) {
                        // the segment's query tile, once the previous segment's score MMAs have read theirs
                        if (nq > 0 && !mbar_wait(&sh->q_free, (nq - 1) & 1, sh, p)) { ok = false; break; }
                        // (a tile past the end of the tree, in the pair form, reads rows that are never stored)
                        mbar_expect_tx(&sh->q_ready, kQTileBytes);
                        for (int h = 0; h < 2; ++h)
                            tma_load_5d(smem_u32(sQ + h * kQHalfBytes), &qmap, h * 64, 0, sg.g,
                                        sg.n0 + (member * kRowsPerCta) / p.G, sg.layer, &sh->q_ready);
                        ++nq;
                    }
                    ids_b[0] = ids_a[0]; ids_b[1] = ids_a[1]; npg_b = npg_a;
                    ids_a[0] = ids[0]; ids_a[1] = ids[1]; npg_a = npg;
                }
            }
            if (sh->abort) {
                // drain: every issued copy must land before the CTA may exit
                for (int n = max(0, rc - kDepth); n < rc; ++n)
                    mbar_wait_quiet(&sh->kv_full[n % kRing], (n / kRing) & 1, p.wait_cycles);
                if (nq > 0) mbar_wait_quiet(&sh->q_ready, (nq - 1) & 1, p.wait_cycles);
            }
        }
    } else if (warp == 10) {
        // =========================== relay (pair form, second CTA) ===========================
        // The MMA thread of the leader waits on the leader's barriers only; what lands in this CTA is passed on
        // to them, in the order in which the MMA thread waits.
        if (kPair && !is_lead && lane == 0) {
            SegIter it;
            it.init(sh);
            Seg sg;
            int rc = 0, nq = 0;
            bool ok = true;
            while (ok && it.next(p, sg)) {
                if (member0 >= sg.rp) continue;
                const int n = sg.s1 - sg.s0;
                for (int i = 0; ok && i < n + 2; ++i) {
                    if (i == 0) {
                        ok = mbar_wait(&sh->q_ready, nq & 1, sh, p);
                        if (!ok) break;
                        ++nq;
                        mbar_arrive_cluster(cluster_addr(&sh->q_ready, 0));
                    }
                    ok = mbar_wait(&sh->kv_full[rc % kRing], (rc / kRing) & 1, sh, p);
                    if (!ok) break;
                    mbar_arrive_cluster(cluster_addr(&sh->kv_full[rc % kRing], 0));
                    ++rc;
                }
            }
        }
    } else if (warp == 9) {
        // =========================== MMA issuer ===========================
        // One thread issues for both slots, in blocks [P V of step i-2, scores of step i]: step i belongs to
        // slot i & 1, so a slot's block runs on the tensor pipe while the other slot's warpgroup is in its
        // softmax, and the blocks never interleave.  The whole instruction stream sits in one single-thread
        // region: a predicated branch around every MMA costs more issue time than the MMA takes to execute.
        if (lane == 0 && is_lead) {
            // descriptors differ only in their 14-bit start-address field (bytes >> 4); shared memory ends below 256 KB
            // (pair form: the same offsets hold the partner's parts in its shared memory)
            const uint32_t dq = desc_lo(smem_u32(sQ), 16);
            const uint32_t dk = desc_lo(smem_u32(sK), 16);
            const uint32_t dv = desc_lo(smem_u32(sV), kTileHalfBytes);
            auto issue_qk = [&](int t, int slot) {
                // S_t = Q K^T: 8 slices of K = 16 over d = 128 (4 per 64-wide half)
                const uint32_t dks = dk + ((slot * kTile) >> 4);
                const uint32_t s_tmem = tmem + t * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t a = dq + (((ks >> 2) * kQHalfBytes + (ks & 3) * 32) >> 4);
                    const uint32_t b = dks + (((ks >> 2) * kKHalf + (ks & 3) * 32) >> 4);
                    if (kPair) mma2_ss(s_tmem, a, b, kDescHi, kIdescQK2, ks > 0 ? 1u : 0u);
                    else mma_ss(s_tmem, a, b, kDescHi, kIdescQK, ks > 0 ? 1u : 0u);
                }
            };
            auto issue_pv = [&](int t, int slot, bool first) {
                // O_t += P_t V: 8 slices of K = 16 keys; P in TMEM (8 columns per slice), V MN-major
                const uint32_t dvs = dv + ((slot * kTile) >> 4);
                const uint32_t s_tmem = tmem + t * 128, o_tmem = tmem + 256 + t * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    if (kPair) mma2_ts(o_tmem, s_tmem + ks * 8, dvs + ((ks * 2048) >> 4), kDescHi, kIdescPV2, (first && ks == 0) ? 0u : 1u);
                    else mma_ts(o_tmem, s_tmem + ks * 8, dvs + ((ks * 2048) >> 4), kDescHi, kIdescPV, (first && ks == 0) ? 0u : 1u);
                }
            };
            SegIter it;
            it.init(sh);
            Seg sg;
            int rc = 0, kc = 0, vc = 0, nseg = 0;           // ring steps, K tiles, V tiles consumed; segments started
            int np[2] = {0, 0};                             // steps of each slot whose probabilities were consumed
            bool ok = true;
            // Every synchronisation instruction costs this thread a couple of hundred clocks, during which
            // at most a few queued MMAs keep the pipe busy: the loop holds as few of them as the protocol
            // allows (one wait and one commit per ring step for the tiles, one of each for the step's slot).
            while (ok && it.next(p, sg)) {
                if (member0 >= sg.rp) continue;
                const int n = sg.s1 - sg.s0;
                ok = mbar_wait<kPair>(&sh->q_ready, nseg & 1, sh, p);
                for (int i = 0; ok && i < n + 2; ++i) {
                    ok = mbar_wait<kPair>(&sh->kv_full[rc % kRing], (rc / kRing) & 1, sh, p);
                    if (!ok) break;
                    const int t = i & 1;
                    if (i >= 2) {
                        // (the warpgroup zeroed the V rows past the end of the sequence before it arrived)
                        ok = mbar_wait<kPair>(&sh->p_full[t], np[t] & 1, sh, p);
                        if (!ok) break;
                        ++np[t];
                        // the segment's first P V products overwrite both accumulators, which the softmax warps
                        // read in the epilogue of the segment before
                        if (i == 2 && nseg > 0) {
                            ok = mbar_wait<kPair>(&sh->epi_done, (nseg - 1) & 1, sh, p);
                            if (!ok) break;
                        }
                        tc_fence_after();
                        issue_pv(t, vc % kStages, i < 4);
                        ++vc;
                        if (i >= n) tc_commit_to<kPair>(&sh->o_full[t]);    // the slot's last step of the segment
                    }
                    if (i < n) {
                        issue_qk(t, kc % kStages);
                        ++kc;
                        tc_commit_to<kPair>(&sh->s_full[t]);
                    }
                    tc_commit_to<kPair>(&sh->kv_done[rc % kRing]);
                    ++rc;
                    if (i == n - 1) tc_commit_to<kPair>(&sh->q_free);   // the segment's last score MMAs read the query tile
                }
                ++nseg;
            }
            if (!ok) {
                // abort: everything this thread has issued must retire before the TMEM and the tiles go away
                tc_commit_to<kPair>(&sh->drain, false);
                mbar_wait_quiet(&sh->drain, 0, p.wait_cycles);
            }
        }
        __syncwarp();
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // =========================== softmax warpgroups ===========================
        // Warpgroup t owns slot t: the steps s0 + t, s0 + t + 2, ... of a segment, with its own score tile S_t,
        // accumulator O_t and running (reference, sum) per row; one thread per query row.  In the epilogue the
        // two slots are combined, warpgroup t taking the output columns [64t, 64t + 64).
        const int t = warp >> 2, q = warp & 3;
        const int r = tid & 127;                        // row inside the tile == TMEM lane
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const uint32_t s_taddr = tmem + lane_base + t * 128;
        const uint32_t o_taddr = tmem + lane_base + 256 + t * 128;
        SegIter it;
        it.init(sh);
        Seg sg;
        int nst = 0;                                    // steps this slot has been through
        int nseg = 0, nseg1 = 0;                        // segments so far; those in which slot 1 had steps
        int rc0 = 0, vc0 = 0;                           // ring steps / V tiles of the CTA before the current segment
        bool ok = true;
        while (ok && it.next(p, sg)) {
            if (member0 >= sg.rp) continue;
            const int M = sg.N * p.G;
            const int n = sg.s1 - sg.s0;
            const int rc_seg = rc0, vc_seg = vc0;       // this segment's first ring step / V tile (= steps so far)
            rc0 += n + 2;
            vc0 += n;
            const int R = member * kRowsPerCta + r;
            const bool row_ok = R < M;
            const int node = row_ok ? R / p.G : 0;
            const bool warp_live = member * kRowsPerCta + q * 32 < M;
            uint64_t anc = 0;
            if (sg.s1 * kStepKeys > sg.L && row_ok) {
                // the segment reaches the tree part: this row's ancestor bitset (the G rows of a node
                // walk the same parent chain, at most N - 1 cached loads deep)
                bool bad = false;
                anc = ancestor_bits(p.parent + sg.n0, sg.N, node, &bad);
                if (bad) { report_status(p.status, SAGE_STATUS_BAD_TREE); anc = 1ull << node; }
            }
            float m_ref = -INFINITY, l_sum = 0.f;
            for (int i = t; i < n; i += 2) {
                const int j = sg.s0 + i;
                ok = mbar_wait(&sh->s_full[t], nst & 1, sh, p);
                if (!ok) break;
                ++nst;
                const int valid = sg.L + sg.N - j * kStepKeys;      // keys of this step that exist
                if (valid < kStepKeys) {
                    // V rows past the end of the sequence may hold anything (a missing second page was not even
                    // copied): zero them so that 0 * V stays 0.  Each warp of the warpgroup takes a quarter of
                    // the rows; the writes are ordered before this warp's arrival, which the P V product waits
                    // for.  The V tile of step s0 + i lands with ring step i + 2 of the segment.
                    const int rcv = rc_seg + i + 2;
                    ok = mbar_wait(&sh->kv_full[rcv % kRing], (rcv / kRing) & 1, sh, p);
                    if (!ok) break;
                    uint8_t* vb = sV + ((vc_seg + i) % kStages) * kTile;
                    constexpr int kChunks = kPair ? 8 : 16;             // 16-byte chunks of a V row held by this CTA
                    for (int c = q * 32 + lane; c < (kStepKeys - valid) * kChunks; c += 128) {
                        const int vr = valid + c / kChunks, ch = c % kChunks;
                        *reinterpret_cast<uint4*>(vb + (ch >> 3) * kTileHalfBytes + vr * 128 + ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
                if (!warp_live) {
                    // none of this warp's 32 rows exists (ragged last tile): keep the barrier protocol
                    // going, leave the probabilities of these rows as they are; their outputs are never stored
                    __syncwarp();
                    if (lane == 0) {
                    if (kPair && !is_lead) mbar_arrive_cluster(lead_p_full[t]);
                    else mbar_arrive(&sh->p_full[t]);
                }
                    continue;
                }
                tc_fence_after();
                const int pos0 = j * kStepKeys;
                const bool masked = pos0 + kStepKeys > sg.L;     // reaches into the tree part (or past the end)
                // the 128 scores of the row: the second half is still on its way while the first is looked at
                uint32_t sr[128];
                tmem_ld32(s_taddr, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
                tmem_ld32(s_taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
                tmem_wait_ld();
                tmem_ld32(s_taddr + 64, *reinterpret_cast<uint32_t(*)[32]>(&sr[64]));
                tmem_ld32(s_taddr + 96, *reinterpret_cast<uint32_t(*)[32]>(&sr[96]));
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (c == 2) tmem_wait_ld();
                    if (masked) mask_chunk(sr + 32 * c, pos0 + 32 * c, sg.L, sg.N, anc);
                    max_chunk(sr + 32 * c, mx);
                }
                // lazy rescale: the reference moves only when the row max grew by more than 2^8 over it
                const float m_cand = mx * p.scale_log2;
                const bool grow = m_cand > m_ref + 8.0f;
                float alpha = 1.0f;
                if (grow) {
                    alpha = fast_exp2(m_ref - m_cand);              // 0 when m_ref was -inf
                    m_ref = m_cand;
                }
                // O_t *= alpha.  The slot's P V product of two steps back has finished: the scores of this step
                // were issued after it, and their completion is what this warp waited for above.
                if (i >= 2 && __any_sync(0xffffffffu, grow)) rescale_o_rows(o_taddr, alpha);
                const float neg_ref = (m_ref == -INFINITY) ? 0.f : -m_ref;
                // probabilities, packed to bf16 in place: chunk c (32 scores) leaves its 16 words at sr[16c ..]
                // (P goes over the first 64 columns of S_t, the first half as soon as it is there)
                uint64_t acc[2] = {0ull, 0ull};
                if (masked) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        exp_chunk<0>(sr + 32 * c, p.scale_log2, neg_ref, sr + 16 * c, acc);   // may hold -inf
                        if (c == 1) tmem_st32(s_taddr, sr);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        exp_chunk<SAGE_EXP2_FMA_PAIRS>(sr + 32 * c, p.scale_log2, neg_ref, sr + 16 * c, acc);
                        if (c == 1) tmem_st32(s_taddr, sr);
                    }
                }
                tmem_st32(s_taddr + 32, sr + 32);
                float sum_a, sum_b;
                f2_unpack(f2_add(acc[0], acc[1]), sum_a, sum_b);
                l_sum = l_sum * alpha + (sum_a + sum_b);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (kPair && !is_lead) mbar_arrive_cluster(lead_p_full[t]);
                    else mbar_arrive(&sh->p_full[t]);
                }
            }
            if (!ok) break;
            // ---- epilogue: the two slots combined, then O / l -> bf16 output, or unnormalised partials for the merge
            const bool has1 = n >= 2;                   // slot 1 took part in this segment
            ok = mbar_wait(&sh->o_full[0], nseg & 1, sh, p);
            if (ok && has1) ok = mbar_wait(&sh->o_full[1], nseg1 & 1, sh, p);
            const uint32_t eseq = (uint32_t)nseg + 1u;
            ++nseg;
            if (has1) ++nseg1;
            if (!ok) break;
            if (warp_live) {
                tc_fence_after();
                // this thread's 64 columns of both accumulators, 32 at a time
                const uint32_t o0 = tmem + lane_base + 256 + 64 * t, o1 = o0 + 128;
                uint32_t oa[32], ob[32];
                tmem_ld32(o0, oa);
                if (has1) tmem_ld32(o1, ob);
                tmem_wait_ld();
                // The row's (reference, sum) of this slot goes to the other warpgroup through two columns of O_t
                // that this thread has just read and nobody else reads: columns 64t and 64t + 1.
                tmem_st2(o_taddr + 64 * t, __float_as_uint(m_ref), __float_as_uint(l_sum));
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    __threadfence_block();
                    sh->eflag[t][q] = eseq;
                }
                // bounded wait for the partner warp (same rows, other slot)
                {
                    volatile uint32_t* flag = &sh->eflag[1 - t][q];
                    bool seen = (*flag == eseq);
                    if (!seen) {
                        const long long t0 = clock64();
                        while (true) {
                            for (int k = 0; k < 64 && !seen; ++k) seen = (*flag == eseq);
                            if (seen || sh->abort) break;
                            if (clock64() - t0 > p.wait_cycles) {
                                raise_abort(sh);
                                report_status(p.status, SAGE_STATUS_TIMEOUT);
                                break;
                            }
                        }
                    }
                    ok = __all_sync(0xffffffffu, seen);
                }
                if (!ok) break;
                tc_fence_after();
                uint32_t pm, pl;
                tmem_ld2(tmem + lane_base + 256 + (1 - t) * 128 + 64 * (1 - t), pm, pl);
                const float m_o = __uint_as_float(pm), l_o = __uint_as_float(pl);
                // weights of the two slots under the common reference (a slot without visible keys has l = 0)
                const float m_all = fmaxf(l_sum > 0.f ? m_ref : -INFINITY, l_o > 0.f ? m_o : -INFINITY);
                const float w_me = l_sum > 0.f ? fast_exp2(m_ref - m_all) : 0.f;
                const float w_ot = l_o > 0.f ? fast_exp2(m_o - m_all) : 0.f;
                const float l_all = l_sum * w_me + l_o * w_ot;
                const bool whole = (sg.s0 == 0 && sg.s1 == sg.steps);
                // factors of O_0 and O_1: the slot weights, and 1 / l for a finished row
                const float inv = whole ? ((l_all > 0.f) ? 1.0f / l_all : 0.f) : 1.0f;
                const float f0 = (t == 0 ? w_me : w_ot) * inv, f1 = has1 ? (t == 0 ? w_ot : w_me) * inv : 0.f;
                __nv_bfloat16* oo = nullptr;
                float* po = nullptr;
                if (whole) {
                    const size_t row = (size_t)(sg.n0 + node) * p.Hq + sg.g * p.G + (row_ok ? R % p.G : 0);
                    oo = p.out + ((size_t)sg.layer * p.sum_nodes * p.Hq + row) * kHeadDim + 64 * t;
                } else {
                    const size_t pr = (((size_t)gang * 2 + (sg.at_range_begin ? 0 : 1)) * p.n_rp + member) * kRowsPerCta + r;
                    po = p.part_o + pr * kHeadDim + 64 * t;
                    if (t == 0 && row_ok) { p.part_ml[pr * 2] = m_all; p.part_ml[pr * 2 + 1] = l_all; }
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    if (c == 1) {
                        tmem_ld32(o0 + 32, oa);
                        if (has1) tmem_ld32(o1 + 32, ob);
                        tmem_wait_ld();
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        float v = __uint_as_float(oa[i]) * f0;
                        if (has1) v = fmaf(__uint_as_float(ob[i]), f1, v);
                        oa[i] = __float_as_uint(v);
                    }
                    if (row_ok) {
                        if (whole) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                uint4 v;
                                v.x = pack_bf16(__uint_as_float(oa[8 * i + 0]), __uint_as_float(oa[8 * i + 1]));
                                v.y = pack_bf16(__uint_as_float(oa[8 * i + 2]), __uint_as_float(oa[8 * i + 3]));
                                v.z = pack_bf16(__uint_as_float(oa[8 * i + 4]), __uint_as_float(oa[8 * i + 5]));
                                v.w = pack_bf16(__uint_as_float(oa[8 * i + 6]), __uint_as_float(oa[8 * i + 7]));
                                *reinterpret_cast<uint4*>(oo + c * 32 + i * 8) = v;
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                *reinterpret_cast<uint4*>(po + c * 32 + i * 4) = make_uint4(oa[4 * i], oa[4 * i + 1], oa[4 * i + 2], oa[4 * i + 3]);
                        }
                    }
                }
            }
            tc_fence_before();                          // the next segment's first P V products overwrite O_0 and O_1
            __syncwarp();
            if (lane == 0) {
                if (kPair && !is_lead) mbar_arrive_cluster(lead_epi_done);
                else mbar_arrive(&sh->epi_done);
            }
        }
    }
    // ---- teardown: every role is past its last TMEM access
    tc_fence_before();
    __syncthreads();
    if (kPair) {
        // neither CTA leaves (or frees tensor memory) while the other may still arrive on its barriers, raise
        // its abort flag, or run MMAs that write its tensor memory
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    if (warp == 9) {
        tc_fence_after();
        if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// Merge of the items that a range boundary cut into segments.  Only a boundary between two gangs'
// ranges can cut an item, so the grid is (x = boundary, y = 32-row chunk): the block finds the item
// its boundary falls into, leaves if the boundary coincides with the item's start or if an earlier
// boundary already lies inside the same item (that block does the work), and otherwise combines the
// item's segments: which gangs hold them, and in which of their two partial slots, follows from
// the positions alone.
__global__ void __launch_bounds__(256) attention_merge_kernel(AttnParams p) {
    __shared__ int s_Wb, s_b, s_s0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_cut = blockIdx.x + 1;                   // boundary between gang k_cut - 1 and gang k_cut
    if (warp == 0) {
        int err = 0, b = 0, s0 = 0;
        const bool mine = schedule_selected(p.select, max_tree_rows(p.node_offsets, p.batch, p.sum_nodes, p.G, lane));
        const int Wb = mine ? steps_per_head(p, lane, &err) : 0;
        if (Wb > 0) {
            const long long W = (long long)p.n_layers * p.Hkv * Wb;
            const int n_act = active_gangs(W, p.n_gangs);
            if (k_cut < n_act) locate(p, lane, (int)(gang_begin(W, n_act, k_cut) % Wb), &b, &s0);
        }
        if (lane == 0) { s_Wb = Wb; s_b = b; s_s0 = s0; }
    }
    __syncthreads();
    const int Wb = s_Wb;
    if (Wb <= 0) return;
    const long long W = (long long)p.n_layers * p.Hkv * Wb;
    const int n_act = active_gangs(W, p.n_gangs);
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
            return (((size_t)k * 2 + slot) * p.n_rp + member) * kRowsPerCta + Rl;
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
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// Tensor maps depend only on (base pointer, shape); a serving loop calls with the same few buffers
// over and over, so the last few encodings are kept.
struct MapKey {
    const void* base;
    long long a, b, c, d;
    int kind;
    bool operator==(const MapKey& o) const {
        return base == o.base && a == o.a && b == o.b && c == o.c && d == o.d && kind == o.kind;
    }
};
constexpr int kMapCache = 16;
static std::mutex g_map_mu;
static MapKey g_map_key[kMapCache];
static CUtensorMap g_map_val[kMapCache];
static int g_map_used = 0, g_map_next = 0;

template <typename Make>
static bool cached_map(CUtensorMap* out, const MapKey& key, Make make) {
    std::lock_guard<std::mutex> lock(g_map_mu);
    for (int i = 0; i < g_map_used; ++i)
        if (g_map_key[i] == key) { *out = g_map_val[i]; return true; }
    if (!make(out)) return false;
    g_map_key[g_map_next] = key;
    g_map_val[g_map_next] = *out;
    g_map_next = (g_map_next + 1) % kMapCache;
    if (g_map_used < kMapCache) ++g_map_used;
    return true;
}

// Pool viewed as [layer][page*Hkv + head][slot][d]; one box = one 64-wide d-half of one (page, head).
static bool make_pool_map(CUtensorMap* map, const void* pool, int n_layers, int n_pages, int n_kv_heads,
                          int64_t layer_stride_elems) {
    const MapKey key{pool, n_layers, n_pages, n_kv_heads, layer_stride_elems, 0};
    return cached_map(map, key, [&](CUtensorMap* m) {
        EncodeTiledFn fn = encode_fn();
        if (!fn) return false;
        const cuuint64_t page_head_bytes = (cuuint64_t)kPageSize * kHeadDim * 2;
        cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)kPageSize, (cuuint64_t)n_pages * n_kv_heads,
                              (cuuint64_t)n_layers};
        cuuint64_t layer_bytes = n_layers > 1 ? (cuuint64_t)layer_stride_elems * 2 : dims[2] * page_head_bytes;
        cuuint64_t strides[3] = {(cuuint64_t)kHeadDim * 2, page_head_bytes, layer_bytes};
        cuuint32_t box[4] = {64, (cuuint32_t)kPageSize, 1, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pool), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// Queries viewed as [layer][node][kv head][head in group][d]; one box = one 64-wide d-half of the
// 128 query rows (128/G nodes x G heads) of a row tile.  Nodes past sum_nodes read as zero.
static bool make_q_map(CUtensorMap* map, const void* q, int n_layers, int sum_nodes, int n_kv_heads, int G) {
    const MapKey key{q, n_layers, sum_nodes, n_kv_heads, G, 1};
    return cached_map(map, key, [&](CUtensorMap* m) {
        EncodeTiledFn fn = encode_fn();
        if (!fn) return false;
        const cuuint64_t row = (cuuint64_t)kHeadDim * 2;
        cuuint64_t dims[5] = {(cuuint64_t)kHeadDim, (cuuint64_t)G, (cuuint64_t)n_kv_heads, (cuuint64_t)sum_nodes,
                              (cuuint64_t)n_layers};
        cuuint64_t strides[4] = {row, row * G, row * G * n_kv_heads, row * G * n_kv_heads * sum_nodes};
        cuuint32_t box[5] = {64, (cuuint32_t)G, 1, (cuuint32_t)(kRowTile / G), 1};
        cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(q), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// One resident CTA per SM (148 when no device can be asked, e.g. a size query on a host without a GPU).
static int resident_ctas() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        (void)cudaGetLastError();
        return 148;
    }
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            return 148;
        }
        cached[dev] = n;
    }
    return cached[dev];
}
// Row tiles of the largest tree the launch can hold.
static int row_tiles(int sum_nodes, int G) {
    const int n = sum_nodes < SAGE_MAX_NODES ? sum_nodes : SAGE_MAX_NODES;      // a tree has at most that many nodes
    return (n * G + kRowTile - 1) / kRowTile;
}

static long long g_wait_cycles = kWaitCyclesDefault;
static int g_producer_off = 0;
static int g_schedule = 0;     // 0: chosen per launch, 1: streaming, 2: split, 3: streaming with CTA pairs

// The split schedule (tree_attention_split.cu).
namespace split {
size_t workspace_size(int n_layers, int batch, int sum_nodes, int n_q_heads, int n_kv_heads, int max_pages_per_seq);
int launch(const void* q, int n_layers, int n_pages, const int32_t* page_table, int max_pages_per_seq,
           const int32_t* seq_len, const int32_t* parent, const int32_t* node_offsets, int batch, int sum_nodes,
           int n_q_heads, int n_kv_heads, float sm_scale, void* out, void* ws, int32_t* status, long long wait_cycles,
           int producer_off, int select, const CUtensorMap& kmap, const CUtensorMap& vmap, cudaStream_t stream);
}  // namespace split

// The streaming schedule for trees of more than one row tile (tree_attention_rows.cu).
namespace rows {
size_t workspace_size(int n_ctas);
int launch(int n_ctas, int select, int n_layers, int n_pages, const int32_t* page_table, int max_pages_per_seq,
           const int32_t* seq_len, const int32_t* parent, const int32_t* node_offsets, int batch, int sum_nodes,
           int n_q_heads, int n_kv_heads, float sm_scale, void* out, void* ws, int32_t* status, long long wait_cycles,
           int producer_off, const CUtensorMap& qmap, const CUtensorMap& kmap, const CUtensorMap& vmap,
           cudaStream_t stream);
}  // namespace rows

// Which schedule runs a launch.
//   streaming: persistent CTAs that walk equal ranges of 128-key steps.  One row tile (up to 128 query rows
//     per KV head): the kernel of this file, single form, which is HBM-bound.  Two row tiles (up to 256 rows):
//     two row tiles per CTA (tree_attention_rows.cu): one CTA holds the whole tree and nothing is read twice.
//   split: grid over (context slice, row pair, layer x sequence x KV head), 64-key steps: wins where the
//     work is tensor-bound (more than 256 rows) and where a launch is too short to give every SM a long
//     stream (single layers, short contexts: fixed costs dominate).
//   pairs: the kernel of this file in its pair form; measured slower than the others everywhere (the
//     hand-overs between the two CTAs lengthen the per-step dependency chain), so never chosen, only forced.
// The host knows how long a launch is, but of the trees only an upper bound: sum_nodes is the size of the
// caller's node arrays, and a decode loop that lives on the device keeps arrays of full capacity whatever
// the trees of a round look like.  So a long launch whose bound allows more than one row tile starts every
// streaming or split kernel that might apply, each told which tree sizes are its own; each works the largest
// tree of the batch out from node_offsets and all but one leave at once (a few microseconds in all).
enum Schedule { kAlternating, kRows, kSplit, kPairs, kOnDevice };
constexpr int kStreamMinSteps = 16;
static Schedule pick_schedule(int n_layers, int batch, int sum_nodes, int n_kv_heads, int G, int max_pages_per_seq) {
    const int tiles = row_tiles(sum_nodes, G);
    if (g_schedule == 1) return tiles == 1 ? kAlternating : kRows;
    if (g_schedule == 2) return kSplit;
    if (g_schedule == 3) return tiles == 1 ? kAlternating : kPairs;
    const long long steps = (long long)n_layers * batch * n_kv_heads * ((max_pages_per_seq + 1) / 2);   // upper bound
    if (steps < (long long)kStreamMinSteps * resident_ctas()) return kSplit;
    return tiles == 1 ? kAlternating : kOnDevice;
}

}  // namespace sage

using namespace sage;

extern "C" size_t sage_tree_attention_workspace_size(int n_layers, int batch, int sum_nodes, int n_q_heads,
                                                     int n_kv_heads, int head_dim, int max_pages_per_seq) {
    if (n_layers < 1 || batch < 1 || sum_nodes < 1 || n_q_heads < 1 || n_kv_heads < 1 || max_pages_per_seq < 1 ||
        n_q_heads % n_kv_heads)
        return 0;
    (void)head_dim;
    // streaming schedules: two partial slots (head and tail of its range) per resident CTA, independent of the
    // problem size; split schedule: one partial per context slice.  Any may run, so the largest is asked for.
    const size_t alternating = (size_t)resident_ctas() * 2 * kRowsPerCta * (kHeadDim + 2) * sizeof(float);
    const size_t rows_ws = rows::workspace_size(resident_ctas());
    const size_t split_ws = split::workspace_size(n_layers, batch, sum_nodes, n_q_heads, n_kv_heads, max_pages_per_seq);
    const size_t streaming = alternating > rows_ws ? alternating : rows_ws;
    return streaming > split_ws ? streaming : split_ws;
}

extern "C" void sage_debug_attention_waits(long long wait_cycles, int producer_off) {
    g_wait_cycles = wait_cycles > 0 ? wait_cycles : kWaitCyclesDefault;
    g_producer_off = producer_off ? 1 : 0;
}

extern "C" void sage_debug_attention_schedule(int schedule) { g_schedule = (schedule >= 1 && schedule <= 3) ? schedule : 0; }

extern "C" int sage_tree_attention(const void* q, const void* k_pool, const void* v_pool, int64_t layer_stride_elems,
                                   int n_layers, int n_pages, const int32_t* page_table, int max_pages_per_seq,
                                   const int32_t* seq_len, const int32_t* parent, const int32_t* node_offsets,
                                   int batch, int sum_nodes, int n_q_heads, int n_kv_heads, int head_dim,
                                   int page_size, float sm_scale, void* out, void* ws, size_t ws_bytes,
                                   int32_t* status, void* stream) {
    if (!q || !k_pool || !v_pool || !page_table || !seq_len || !parent || !node_offsets || !out)
        return SAGE_ERR_INVALID_ARG;
    if (n_layers < 1 || n_pages < 1 || max_pages_per_seq < 1 || batch < 0 || sum_nodes < 1 || n_q_heads < 1 ||
        n_kv_heads < 1 || layer_stride_elems < 0 || !(sm_scale > 0.f))
        return SAGE_ERR_INVALID_ARG;
    if (head_dim != kHeadDim || page_size != kPageSize) return SAGE_ERR_UNSUPPORTED;
    if (n_q_heads % n_kv_heads) return SAGE_ERR_UNSUPPORTED;
    const int G = n_q_heads / n_kv_heads;
    if (G != 1 && G != 2 && G != 4 && G != 8) return SAGE_ERR_UNSUPPORTED;
    if ((long long)n_layers * batch * n_kv_heads > 0x7fffffffll || max_pages_per_seq > (1 << 24)) return SAGE_ERR_UNSUPPORTED;
    if ((((uintptr_t)q | (uintptr_t)k_pool | (uintptr_t)v_pool | (uintptr_t)out) & 15) || (layer_stride_elems & 7))
        return SAGE_ERR_INVALID_ARG;
    if (n_layers > 1 && layer_stride_elems < (int64_t)n_pages * n_kv_heads * kPageSize * kHeadDim)
        return SAGE_ERR_INVALID_ARG;
    if (batch == 0) return SAGE_OK;
    const size_t need = sage_tree_attention_workspace_size(n_layers, batch, sum_nodes, n_q_heads, n_kv_heads,
                                                           head_dim, max_pages_per_seq);
    if (!ws || ws_bytes < need || ((uintptr_t)ws & 15)) return SAGE_ERR_WORKSPACE;
    const Schedule sched = pick_schedule(n_layers, batch, sum_nodes, n_kv_heads, G, max_pages_per_seq);
    if (sched == kSplit && (long long)n_layers * batch * n_kv_heads > 65535) return SAGE_ERR_UNSUPPORTED;    // its grid limit
    CUtensorMap qmap, kmap, vmap;
    if (!make_pool_map(&kmap, k_pool, n_layers, n_pages, n_kv_heads, layer_stride_elems) ||
        !make_pool_map(&vmap, v_pool, n_layers, n_pages, n_kv_heads, layer_stride_elems))
        return SAGE_ERR_CUDA;
    if (sched == kSplit)
        return split::launch(q, n_layers, n_pages, page_table, max_pages_per_seq, seq_len, parent, node_offsets, batch,
                             sum_nodes, n_q_heads, n_kv_heads, sm_scale, out, ws, status, g_wait_cycles, g_producer_off,
                             0, kmap, vmap, as_stream(stream));
    if (!make_q_map(&qmap, q, n_layers, sum_nodes, n_kv_heads, G)) return SAGE_ERR_CUDA;
    if (sched == kRows)
        return rows::launch(resident_ctas(), 0, n_layers, n_pages, page_table, max_pages_per_seq, seq_len, parent,
                            node_offsets, batch, sum_nodes, n_q_heads, n_kv_heads, sm_scale, out, ws, status,
                            g_wait_cycles, g_producer_off, qmap, kmap, vmap, as_stream(stream));
    const int tiles = row_tiles(sum_nodes, G);
    if (sched == kOnDevice) {
        // the kernels for two row tiles and (if the bound allows them) for more; the one for one row tile follows below
        int rc = rows::launch(resident_ctas(), 2, n_layers, n_pages, page_table, max_pages_per_seq, seq_len, parent,
                              node_offsets, batch, sum_nodes, n_q_heads, n_kv_heads, sm_scale, out, ws, status,
                              g_wait_cycles, g_producer_off, qmap, kmap, vmap, as_stream(stream));
        if (rc != SAGE_OK) return rc;
        if (tiles > 2) {
            if ((long long)n_layers * batch * n_kv_heads > 65535) return SAGE_ERR_UNSUPPORTED;    // grid limit of the split schedule
            rc = split::launch(q, n_layers, n_pages, page_table, max_pages_per_seq, seq_len, parent, node_offsets, batch,
                               sum_nodes, n_q_heads, n_kv_heads, sm_scale, out, ws, status, g_wait_cycles,
                               g_producer_off, 3, kmap, vmap, as_stream(stream));
            if (rc != SAGE_OK) return rc;
        }
    }
    const int n_ctas = resident_ctas();
    AttnParams p{};
    // one row tile: single CTAs; more (pair form only): CTA pairs, two row tiles each
    const bool pair = sched == kPairs;
    p.n_rp = pair ? 2 * ((tiles + 1) / 2) : 1;
    p.n_gangs = n_ctas / p.n_rp;
    p.out = (__nv_bfloat16*)out;
    p.part_o = (float*)ws;
    p.part_ml = (float*)ws + (size_t)n_ctas * 2 * kRowsPerCta * kHeadDim;
    p.page_table = page_table; p.seq_len = seq_len; p.parent = parent; p.node_offsets = node_offsets;
    p.status = status;
    p.n_layers = n_layers; p.batch = batch; p.sum_nodes = sum_nodes; p.n_pages = n_pages;
    p.max_pages = max_pages_per_seq; p.Hq = n_q_heads; p.Hkv = n_kv_heads; p.G = G;
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.wait_cycles = g_wait_cycles;
    p.producer_off = g_producer_off;
    p.select = sched == kOnDevice ? 1 : 0;

    // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SAGE_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(tree_attention_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(tree_attention_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
            return SAGE_ERR_CUDA;
        attr_set[dev] = true;
    }
    if (pair) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(p.n_gangs * p.n_rp));
        cfg.blockDim = dim3(kAttnThreads);
        cfg.dynamicSmemBytes = kSmemBytes;
        cfg.stream = as_stream(stream);
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, tree_attention_kernel<true>, p, qmap, kmap, vmap) != cudaSuccess) return SAGE_ERR_CUDA;
    } else {
        tree_attention_kernel<false><<<p.n_gangs * p.n_rp, kAttnThreads, kSmemBytes, as_stream(stream)>>>(p, qmap, kmap, vmap);
    }
    if (p.n_gangs > 1) {
        dim3 mg((unsigned)(p.n_gangs - 1), (unsigned)((p.n_rp * kRowsPerCta + 31) / 32));
        attention_merge_kernel<<<mg, 256, 0, as_stream(stream)>>>(p);
    }
    return launch_status();
}
