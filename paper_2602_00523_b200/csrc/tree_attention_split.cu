// Tree-masked verification attention over a paged bf16 KV cache (Section 2.2;
// Algorithm 1, the target pass over all tree tokens; Section 3.3 Phase 2), sm_100a:
// the split schedule, used for launches that are tensor-bound (more than 256 query rows
// per KV head) or too small to give every SM a long stream of work (single layers,
// short contexts).  tree_attention.cu holds the dispatch and, with tree_attention_rows.cu, the
// streaming schedule.
//
// Flash-decoding layout.  The N tree nodes x G query heads that share one KV head
// form M = N*G query rows (<= 512).  A CTA owns up to two 128-row tiles of them and
// one slice of the context (split-K).  The pipeline step is one 64-token page:
//   TMA      : K and V pages -> 128B-swizzled shared memory, two 5-page rings, mbarriers
//   tcgen05  : S_t = Q_t K^T (128 x 64, fp32) into TMEM; one warp per row tile issues, through
//              one elected lane, with warp-uniform descriptor arithmetic
//   softmax  : one warpgroup per row tile, one thread per row: tcgen05.ld S, online
//              softmax in fp32 (log2 domain, lazy rescale), P -> bf16 back into TMEM
//   tcgen05  : O_t += P_t V with P as the TMEM A operand, V MN-major from shared memory
// Every row tile has two S buffers (even / odd pages), so the tensor pipe computes the
// scores of page j+1 while the warpgroup is busy with page j and never waits for it.
// TMEM map (512 columns): tile t owns S_t,even [128t, 128t+64), S_t,odd [128t+64, 128t+128)
// (P overlays the first 32 columns of its S buffer) and O_t [256+128t, 384+128t).
// Slices are merged by attention_split_merge_kernel (warp per output row).  All waits are
// bounded: on expiry the CTA records SAGE_STATUS_TIMEOUT, drains its copies, frees its
// TMEM and returns.
#include <cuda.h>

#include "sage_common.cuh"

namespace sage {
namespace split {

constexpr int kRowTile = 128;                  // query rows per MMA tile
constexpr int kRowsPerCta = 2 * kRowTile;
constexpr int kStages = 5;                     // depth of the K ring and of the V ring, in pages
constexpr int kPageBytes = kPageSize * kHeadDim * 2;        // one (page, head) tile: 16 KB
constexpr int kPageHalfBytes = kPageSize * 64 * 2;          // one 64-wide d-half of a page: 8 KB
constexpr int kQTileBytes = kRowTile * kHeadDim * 2;        // 32 KB
constexpr int kQHalfBytes = kRowTile * 64 * 2;              // one 64-wide d-half of a Q tile: 16 KB
constexpr int kAttnThreads = 352;              // 2 softmax warpgroups + TMA warp + one MMA warp per row tile
constexpr int kSmemBytes = 2 * kQTileBytes + 2 * kStages * kPageBytes + 1024 /*align*/ + 512 /*barriers*/;

struct AttnParams {
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    float* part_o;     // [layer][split][sum_nodes*Hq][128]   unnormalised
    float* part_ml;    // [layer][split][sum_nodes*Hq][2]     (reference max in log2 units, l)
    const int32_t* page_table;
    const int32_t* seq_len;
    const int32_t* parent;
    const int32_t* node_offsets;
    int32_t* status;
    int n_layers, batch, sum_nodes, n_pages, max_pages;
    int Hq, Hkv, G, n_splits;
    float scale_log2;  // sm_scale * log2(e)
    long long wait_cycles;     // budget of every on-device wait
    int producer_off;          // diagnostics: the TMA warp issues no copies (every consumer wait then runs out)
    int select;                // which tree sizes this launch is for (schedule_selected)
};

struct __align__(8) Barriers {
    uint64_t k_full[kStages], k_empty[kStages];
    uint64_t v_full[kStages], v_empty[kStages];
    uint64_t s_full[2][2];     // [row tile][page parity]: scores of a page are in TMEM
    uint64_t p_full[2][2];     // [row tile][page parity]: probabilities of a page are in TMEM
    uint64_t pv_done[2];       // [row tile]: completes once per page, when its P V product has finished
    uint64_t o_full[2];        // [row tile]: every MMA of the tile has finished
    uint64_t q_ready;          // the query tiles are staged in shared memory
    uint32_t tmem_base;
    volatile int abort;
};
static_assert(sizeof(Barriers) <= 512, "barrier block outgrew its shared-memory reservation");

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
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Barriers* bars, int32_t* status, long long budget) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity)) return true;
        if (bars->abort) return false;
        if (clock64() - t0 > budget) {
            bars->abort = 1;
            report_status(status, SAGE_STATUS_TIMEOUT);
            return false;
        }
    }
}

// ---- TMA ----------------------------------------------------------------------
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar)) : "memory");
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
// D[tmem] (+)= A[smem desc] * B[smem desc]
template <bool kAcc>
__device__ __forceinline__ void mma_ss(bool leader, uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
    if (leader)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "n"(kAcc ? 1 : 0) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void mma_ts(bool leader, uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    if (leader)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
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
// offsets in 16-byte units, version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: D fp32, A and B bf16, M = 128, N as given.
constexpr uint32_t idesc_f16(uint32_t n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
constexpr uint32_t kIdescQK = idesc_f16(kPageSize);              // S (128 x 64): A, B both K-major
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

// One 64-key half of a softmax step for one query row: p = 2^(s * scale + neg_ref), packed to
// bf16 pairs (in place, over the first 32 words of `sr`), and their fp32 sum.  kEmu of every 8
// column pairs take the FMA-pipe exp2.  Written in stages over the whole row so that neighbouring
// instructions are independent: a softmax warp mostly runs alone on its scheduler.
template <int kEmu>
__device__ __forceinline__ float softmax_half(uint32_t (&sr)[64], float scale, float neg_ref) {
    const uint64_t scale2 = f2_pack(scale, scale), nref2 = f2_pack(neg_ref, neg_ref);
    uint64_t x2[32];
#pragma unroll
    for (int i = 0; i < 32; ++i)
        x2[i] = f2_fma(f2_pack(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1])), scale2, nref2);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        float p0, p1;
        if ((i & 7) < kEmu) {
            exp2_pair_fma(x2[i], p0, p1);
        } else {
            float x0, x1;
            f2_unpack(x2[i], x0, x1);
            p0 = fast_exp2(x0);
            p1 = fast_exp2(x1);
        }
        x2[i] = f2_pack(p0, p1);
    }
    uint64_t acc[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = x2[i];
#pragma unroll
    for (int i = 4; i < 32; ++i) acc[i & 3] = f2_add(acc[i & 3], x2[i]);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        float p0, p1;
        f2_unpack(x2[i], p0, p1);
        sr[i] = pack_bf16(p0, p1);
    }
    float a, b;
    f2_unpack(f2_add(f2_add(acc[0], acc[1]), f2_add(acc[2], acc[3])), a, b);
    return a + b;
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

#ifndef SAGE_EXP2_FMA_PAIRS
#define SAGE_EXP2_FMA_PAIRS 1       // of every 8 column pairs (measured best with both warpgroups busy at once)
#endif

__global__ void __launch_bounds__(kAttnThreads, 1)
tree_attention_split_kernel(const AttnParams p, const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_anc[SAGE_MAX_NODES];
    __shared__ int32_t s_parent[SAGE_MAX_NODES];
    __shared__ int s_flag;
    // 1024-byte alignment: the 128B swizzle pattern repeats every 1024 bytes of address
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                                 // [2 tiles][2 d-halves][128 rows][128 B]
    uint8_t* sK = smem + 2 * kQTileBytes;               // [kStages][2 d-halves][64 keys][128 B]
    uint8_t* sV = sK + kStages * kPageBytes;            // [kStages][2 d-halves][64 keys][128 B]
    Barriers* bars = reinterpret_cast<Barriers*>(sV + kStages * kPageBytes);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, rpair = blockIdx.y;
    const int g = blockIdx.z % p.Hkv;
    const int b = (blockIdx.z / p.Hkv) % p.batch;
    const int layer = blockIdx.z / (p.Hkv * p.batch);

    // ---- uniform early exits (before any barrier or TMEM is touched)
    // (every warp works the batch's largest tree out for itself: the same answer everywhere, no barrier)
    if (p.select != 0 && !schedule_selected(p.select, max_tree_rows(p.node_offsets, p.batch, p.sum_nodes, p.G, lane))) return;
    const int n0 = p.node_offsets[b];
    const int N = p.node_offsets[b + 1] - n0;
    const int L = p.seq_len[b];
    if (N < 1 || N > SAGE_MAX_NODES || n0 < 0 || n0 + N > p.sum_nodes) {
        if (tid == 0) report_status(p.status, SAGE_STATUS_BAD_TREE);
        return;
    }
    const int T = L + N;
    if (L < 0 || T > p.max_pages * kPageSize) {
        if (tid == 0) report_status(p.status, SAGE_STATUS_BAD_PAGE);
        return;
    }
    const int M = N * p.G;
    if (rpair * kRowsPerCta >= M) return;
    const int n_rtiles = (M - rpair * kRowsPerCta > kRowTile) ? 2 : 1;

    // this CTA's slice of the context, in pages
    const int n_pages_seq = (T + kPageSize - 1) / kPageSize;
    const int per_split = (n_pages_seq + p.n_splits - 1) / p.n_splits;
    const int pg_begin = split * per_split;
    const int pg_end = min(n_pages_seq, pg_begin + per_split);
    const int ns = max(0, pg_end - pg_begin);           // pipeline steps
    const int32_t* pages = p.page_table + (size_t)b * p.max_pages + pg_begin;
    // One round of global loads: the parent array goes to shared memory (the ancestor walks below
    // would otherwise be chains of dependent global loads), and the page ids of this slice are
    // checked before the TMA warp uses them as coordinates.
    if (tid == 0) s_flag = 0;
    if (tid < SAGE_MAX_NODES) s_parent[tid] = (tid < N) ? p.parent[n0 + tid] : -1;
    bool bad_page = false;
    for (int j = tid; j < ns; j += kAttnThreads) {
        const int id = pages[j];
        if (id < 0 || id >= p.n_pages) bad_page = true;
    }
    __syncthreads();
    if (bad_page) s_flag = 2;
    if (tid < SAGE_MAX_NODES) {
        uint64_t a = 0;
        if (tid < N) {
            bool bad = false;
            a = ancestor_bits(s_parent, N, tid, &bad);
            if (bad) { s_flag = 1; a = 1ull << tid; }
        }
        s_anc[tid] = a;
    }
    __syncthreads();
    if (s_flag) {
        if (tid == 0) report_status(p.status, s_flag == 1 ? SAGE_STATUS_BAD_TREE : SAGE_STATUS_BAD_PAGE);
        return;
    }

    // ---- set-up: barriers, TMEM, Q tiles
    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&bars->k_full[i], 1); mbar_init(&bars->k_empty[i], n_rtiles);   // one release per MMA warp
            mbar_init(&bars->v_full[i], 1); mbar_init(&bars->v_empty[i], n_rtiles);
        }
        for (int t = 0; t < 2; ++t) {
            for (int x = 0; x < 2; ++x) { mbar_init(&bars->s_full[t][x], 1); mbar_init(&bars->p_full[t][x], 4); }
            mbar_init(&bars->pv_done[t], 1);
            mbar_init(&bars->o_full[t], 1);
        }
        mbar_init(&bars->q_ready, 8);
        bars->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&bars->tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // From here the TMA producer streams K/V while the softmax warps stage the query tiles.
    if (warp < 8) {
        // Q rows -> K-major 128B-swizzled tiles; rows past M are zero.  Eight 16-byte loads are in
        // flight per thread before the first store (the loads are latency-bound otherwise).
        for (int c0 = tid; c0 < n_rtiles * kRowTile * 16; c0 += 256 * 8) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u * 256;
                const int t = c / (kRowTile * 16), r = (c / 16) % kRowTile, ch = c % 16;
                const int R = rpair * kRowsPerCta + t * kRowTile + r;
                v[u] = make_uint4(0, 0, 0, 0);
                if (R < M) {
                    const size_t row = ((size_t)layer * p.sum_nodes + n0 + R / p.G) * p.Hq + g * p.G + R % p.G;
                    v[u] = *reinterpret_cast<const uint4*>(p.q + row * kHeadDim + ch * 8);
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u * 256;
                const int t = c / (kRowTile * 16), r = (c / 16) % kRowTile, ch = c % 16;
                const int half = ch >> 3, cc = ch & 7;
                *reinterpret_cast<uint4*>(sQ + t * kQTileBytes + half * kQHalfBytes + r * 128 + ((cc ^ (r & 7)) << 4)) = v[u];
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA unit
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->q_ready);
    }
    const uint32_t tmem = bars->tmem_base;

    if (warp == 8) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            int issued_k = 0, issued_v = 0;
            for (int j = 0; j < ns && !p.producer_off; ++j) {
                const int slot = j % kStages, use = j / kStages;
                const int c2 = pages[j] * p.Hkv + g;
                if (use > 0 && !mbar_wait(&bars->k_empty[slot], (use - 1) & 1, bars, p.status, p.wait_cycles)) break;
                mbar_expect_tx(&bars->k_full[slot], kPageBytes);
                for (int h = 0; h < 2; ++h)
                    tma_load_4d(smem_u32(sK + slot * kPageBytes + h * kPageHalfBytes), &kmap, h * 64, 0, c2, layer,
                                &bars->k_full[slot]);
                issued_k = j + 1;
                if (use > 0 && !mbar_wait(&bars->v_empty[slot], (use - 1) & 1, bars, p.status, p.wait_cycles)) break;
                mbar_expect_tx(&bars->v_full[slot], kPageBytes);
                for (int h = 0; h < 2; ++h)
                    tma_load_4d(smem_u32(sV + slot * kPageBytes + h * kPageHalfBytes), &vmap, h * 64, 0, c2, layer,
                                &bars->v_full[slot]);
                issued_v = j + 1;
            }
            if (bars->abort) {
                // drain: every issued copy must land before the CTA may exit
                for (int n = max(0, issued_k - kStages); n < issued_k; ++n) {
                    const long long t0 = clock64();
                    while (!mbar_try(&bars->k_full[n % kStages], (n / kStages) & 1) && clock64() - t0 < p.wait_cycles) {}
                }
                for (int n = max(0, issued_v - kStages); n < issued_v; ++n) {
                    const long long t0 = clock64();
                    while (!mbar_try(&bars->v_full[n % kStages], (n / kStages) & 1) && clock64() - t0 < p.wait_cycles) {}
                }
            }
        }
    } else if (warp >= 9) {
        // =========================== MMA issuers: warp 9 -> row tile 0, warp 10 -> row tile 1 ===========================
        // Broadcasts from lane 0 tell the compiler that these values are warp-uniform, so that the
        // descriptor arithmetic and the loop control below can stay in the uniform datapath.
        const int t = __shfl_sync(0xffffffffu, warp - 9, 0);
        const uint32_t tmem = __shfl_sync(0xffffffffu, bars->tmem_base, 0);
        const int ns = __shfl_sync(0xffffffffu, max(0, pg_end - pg_begin), 0);
        const int n_rtiles = __shfl_sync(0xffffffffu, (M - rpair * kRowsPerCta > kRowTile) ? 2 : 1, 0);
        const int first_pos = __shfl_sync(0xffffffffu, pg_begin * kPageSize, 0);
        const int T = __shfl_sync(0xffffffffu, L + N, 0);
        const bool leader = elect_one();
        // lane 0 polls, the result is broadcast so that the warp never diverges on a wait
        auto wait_all = [&](uint64_t* bar, uint32_t parity) {
            int r = 1;
            if (lane == 0) r = mbar_wait(bar, parity, bars, p.status, p.wait_cycles) ? 1 : 0;
            return __shfl_sync(0xffffffffu, r, 0) != 0;
        };
        // descriptors differ only in their 14-bit start-address field (bytes >> 4); shared memory ends below 256 KB
        const uint64_t dq = make_desc(smem_u32(sQ) + t * kQTileBytes, 16, 1024);
        const uint64_t dk = make_desc(smem_u32(sK), 16, 1024);
        const uint64_t dv = make_desc(smem_u32(sV), kPageHalfBytes, 1024);
        const uint32_t s_tmem = tmem + t * 128, o_tmem = tmem + 256 + t * 128;
        auto issue_qk = [&](int x, int slot) {
            // S_t,x = Q_t K^T: 8 steps of K = 16 over d = 128 (4 per 64-wide half)
            const uint64_t dks = dk + (uint64_t)((slot * kPageBytes) >> 4);
            const uint32_t d = s_tmem + x * 64;
            mma_ss<false>(leader, d, dq, dks, kIdescQK);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                mma_ss<true>(leader, d, dq + (uint64_t)(((ks >> 2) * kQHalfBytes + (ks & 3) * 32) >> 4),
                             dks + (uint64_t)(((ks >> 2) * kPageHalfBytes + (ks & 3) * 32) >> 4), kIdescQK);
        };
        auto issue_pv = [&](int x, int slot, bool first) {
            // O_t += P_t,x V: 4 steps of K = 16 keys; P in TMEM (8 columns per step), V MN-major
            const uint64_t dvs = dv + (uint64_t)((slot * kPageBytes) >> 4);
            const uint32_t a = s_tmem + x * 64;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                mma_ts(leader, o_tmem, a + ks * 8, dvs + (uint64_t)((ks * 2048) >> 4), kIdescPV, (!first || ks > 0) ? 1u : 0u);
        };
        bool ok = ns > 0 && t < n_rtiles;
        if (ok) ok = wait_all(&bars->q_ready, 0);
        // prologue: scores of the first two pages
        for (int j = 0; ok && j < min(2, ns); ++j) {
            ok = wait_all(&bars->k_full[j], 0);
            if (!ok) break;
            tc_fence_after();
            issue_qk(j, j);
            tc_commit(leader, &bars->s_full[t][j]);
            tc_commit(leader, &bars->k_empty[j]);
        }
        // The V page of step j and the K page of step j+2 are looked up one step ahead (`stage_inputs`),
        // while the softmax of the previous page is still running, so that only the wait for the
        // probabilities sits between the softmax and the MMAs that depend on it.
        auto stage_inputs = [&](int j) -> bool {
            if (j >= ns) return true;
            const int vslot = j % kStages;
            if (!wait_all(&bars->v_full[vslot], (j / kStages) & 1)) return false;
            const int valid = min(kPageSize, T - first_pos - j * kPageSize);
            if (valid < kPageSize) {
                // rows past the end of the sequence may hold anything: zero them so that 0 * V stays 0
                // (both MMA warps write the same zeros; each orders its own writes before its own MMAs)
                uint8_t* vb = sV + vslot * kPageBytes;
                for (int c = lane; c < (kPageSize - valid) * 16; c += 32) {
                    const int r = valid + c / 16, ch = c % 16;
                    *reinterpret_cast<uint4*>(vb + (ch >> 3) * kPageHalfBytes + r * 128 + ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
            }
            const int jn = j + 2;
            if (jn < ns && !wait_all(&bars->k_full[jn % kStages], (jn / kStages) & 1)) return false;
            return true;
        };
        if (ok) ok = stage_inputs(0);
        for (int j = 0; ok && j < ns; ++j) {
            const int x = j & 1, vslot = j % kStages;
            const int jn = j + 2, kslot = jn % kStages;
            ok = wait_all(&bars->p_full[t][x], (j >> 1) & 1);
            if (!ok) break;
            tc_fence_after();
            issue_pv(x, vslot, j == 0);
            tc_commit(leader, &bars->pv_done[t]);
            tc_commit(leader, &bars->v_empty[vslot]);
            if (jn < ns) {
                // the scores of page j+2 reuse this S buffer: in pipe order after P V of page j
                issue_qk(x, kslot);
                tc_commit(leader, &bars->s_full[t][x]);
                tc_commit(leader, &bars->k_empty[kslot]);
            }
            ok = stage_inputs(j + 1);
        }
        if (t < n_rtiles) tc_commit(leader, &bars->o_full[t]);     // arrives when every MMA of this tile has completed
        if (!ok && t < n_rtiles && lane == 0) {
            // abort: everything this warp has issued must retire before the TMEM and the tiles go away
            const long long t0 = clock64();
            while (!mbar_try(&bars->o_full[t], 0) && clock64() - t0 < p.wait_cycles) {}
        }
        __syncwarp();
    } else {
        // =========================== softmax warpgroups ===========================
        const int t = warp >> 2;                        // row tile of this warpgroup
        const int r = tid & 127;                        // row inside the tile == TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_taddr = tmem + lane_base + t * 128;
        const uint32_t o_taddr = tmem + lane_base + 256 + t * 128;
        const int R = rpair * kRowsPerCta + t * kRowTile + r;
        const bool row_ok = R < M;
        const int node = row_ok ? R / p.G : 0;
        const uint64_t anc = s_anc[node];
        const bool warp_live = rpair * kRowsPerCta + t * kRowTile + (warp & 3) * 32 < M;
        float m_ref = -INFINITY, l_sum = 0.f;
        bool ok = (t < n_rtiles);
        for (int j = 0; ok && j < ns; ++j) {
            const int x = j & 1;
            ok = mbar_wait(&bars->s_full[t][x], (j >> 1) & 1, bars, p.status, p.wait_cycles);
            if (!ok) break;
            if (!warp_live) {
                // none of this warp's 32 rows exists (ragged last tile): keep the barrier protocol
                // going, leave the probabilities of these rows as they are; their outputs are never stored
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->p_full[t][x]);
                continue;
            }
            tc_fence_after();
            uint32_t sr[64];
            tmem_ld32(s_taddr + x * 64, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
            tmem_ld32(s_taddr + x * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
            tmem_wait_ld();
            const int pos0 = (pg_begin + j) * kPageSize;
            const bool masked = pos0 + kPageSize > L;
            if (masked) {
                // page reaches into the tree part (or past the end): apply the ancestor mask
#pragma unroll
                for (int i = 0; i < 64; ++i) {
                    const int jt = pos0 + i - L;                      // tree slot; < 0 = prefix
                    const bool vis = jt < 0 || (jt < N && ((anc >> jt) & 1ull));
                    if (!vis) sr[i] = 0xff800000u;                    // -inf
                }
            }
            // row max: eight independent chains of three-input max
            float mx8[8];
#pragma unroll
            for (int q8 = 0; q8 < 8; ++q8) {
                float mq = max3(__uint_as_float(sr[q8 * 8]), __uint_as_float(sr[q8 * 8 + 1]), __uint_as_float(sr[q8 * 8 + 2]));
                mq = max3(mq, __uint_as_float(sr[q8 * 8 + 3]), __uint_as_float(sr[q8 * 8 + 4]));
                mq = max3(mq, __uint_as_float(sr[q8 * 8 + 5]), __uint_as_float(sr[q8 * 8 + 6]));
                mx8[q8] = fmaxf(mq, __uint_as_float(sr[q8 * 8 + 7]));
            }
            const float mx = fmaxf(max3(mx8[0], mx8[1], mx8[2]), fmaxf(max3(mx8[3], mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
            const float m_cand = mx * p.scale_log2;
            // lazy rescale: move the reference only when the row max grew by more than 2^8
            const bool grow = m_cand > m_ref + 8.0f;
            float alpha = 1.0f;
            if (grow) {
                alpha = fast_exp2(m_ref - m_cand);          // 0 when m_ref was -inf
                m_ref = m_cand;
            }
            const float neg_ref = (m_ref == -INFINITY) ? 0.f : -m_ref;
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
                // O_t *= alpha, once the P V product of page j-1 has finished
                ok = mbar_wait(&bars->pv_done[t], (j - 1) & 1, bars, p.status, p.wait_cycles);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                rescale_o_rows(o_taddr, alpha);
            }
            float sum;
            if (masked) sum = softmax_half<0>(sr, p.scale_log2, neg_ref);     // may hold -inf
            else sum = softmax_half<SAGE_EXP2_FMA_PAIRS>(sr, p.scale_log2, neg_ref);
            tmem_st32(s_taddr + x * 64, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));   // P over the first 32 columns of this S buffer
            l_sum = l_sum * alpha + sum;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->p_full[t][x]);
        }
        // ---- epilogue: O_t / l -> bf16 output, or unnormalised partials for the merge
        if (t < n_rtiles) {
            if (ns > 0 && ok) ok = mbar_wait(&bars->o_full[t], 0, bars, p.status, p.wait_cycles);
            if (ok) tc_fence_after();
            const size_t rows_total = (size_t)p.sum_nodes * p.Hq;
            const size_t row = (size_t)(n0 + node) * p.Hq + g * p.G + (row_ok ? R % p.G : 0);
            const float inv = (l_sum > 0.f) ? 1.0f / l_sum : 0.f;
            float* po = nullptr;
            __nv_bfloat16* oo = nullptr;
            if (p.n_splits == 1) {
                oo = p.out + ((size_t)layer * rows_total + row) * kHeadDim;
            } else {
                const size_t pr = ((size_t)layer * p.n_splits + split) * rows_total + row;
                po = p.part_o + pr * kHeadDim;
                if (row_ok && ok) { p.part_ml[pr * 2] = m_ref; p.part_ml[pr * 2 + 1] = (ns > 0) ? l_sum : 0.f; }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t orr[32];
                if (ns > 0 && ok) {
                    tmem_ld32(o_taddr + c * 32, orr);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) orr[i] = 0u;
                }
                if (row_ok && ok) {
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
    }
    // ---- teardown: every role is past its last TMEM access
    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// Split-K merge: one warp per (layer, node, head) row.  Lanes first reduce (m, l) over
// the slices with shuffles, then each lane combines its four output columns.
__global__ void attention_split_merge_kernel(AttnParams p) {
    const int warps = blockDim.x >> 5;
    const size_t rows_total = (size_t)p.sum_nodes * p.Hq;
    const size_t row = (size_t)blockIdx.x * warps + (threadIdx.x >> 5);
    const int layer = blockIdx.y;
    const int lane = threadIdx.x & 31;
    if (p.select != 0 && !schedule_selected(p.select, max_tree_rows(p.node_offsets, p.batch, p.sum_nodes, p.G, lane))) return;
    if (row >= rows_total) return;
    const int node = (int)(row / p.Hq);
    if (node >= p.node_offsets[p.batch]) return;       // rows past the live nodes were never written
    float m = -INFINITY, l = 0.f;
    if (lane < p.n_splits) {
        const size_t r = ((size_t)layer * p.n_splits + lane) * rows_total + row;
        m = p.part_ml[r * 2];
        l = p.part_ml[r * 2 + 1];
    }
    float mx = (l > 0.f) ? m : -INFINITY;
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float w = (l > 0.f) ? exp2f(m - mx) : 0.f;   // weight of this lane's slice
    float lsum = l * w;
    for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < p.n_splits; ++s) {
        const float ws = __shfl_sync(0xffffffffu, w, s);
        if (ws == 0.f) continue;
        const size_t r = ((size_t)layer * p.n_splits + s) * rows_total + row;
        const float4 v = reinterpret_cast<const float4*>(p.part_o + r * kHeadDim)[lane];
        acc.x = fmaf(ws, v.x, acc.x); acc.y = fmaf(ws, v.y, acc.y);
        acc.z = fmaf(ws, v.z, acc.z); acc.w = fmaf(ws, v.w, acc.w);
    }
    const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
    reinterpret_cast<uint2*>(p.out + ((size_t)layer * rows_total + row) * kHeadDim)[lane] = packed;
}

static int row_pairs_for(int sum_nodes, int G) {
    const int n = sum_nodes < SAGE_MAX_NODES ? sum_nodes : SAGE_MAX_NODES;      // a tree has at most that many nodes
    return (n * G + kRowsPerCta - 1) / kRowsPerCta;
}

static int pick_splits(int n_layers, int batch, int n_kv_heads, int G, int max_pages, int sum_nodes) {
    // One CTA is resident per SM.  Take the smallest slice count whose CTA count fills whole
    // waves of 148 SMs to >= 90 % (else the best one), keeping >= 4 pages per slice (short contexts are latency-bound:
    // more, shorter slices beat fewer CTAs with longer loops; measured at 2k context).
    const long base = (long)n_layers * batch * n_kv_heads * row_pairs_for(sum_nodes, G);
    int s_max = max_pages / 4;
    if (s_max > 32) s_max = 32;
    if (s_max < 1) s_max = 1;
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= s_max; ++s) {
        const long ctas = base * s;
        const double eff = (double)ctas / (148.0 * ((ctas + 147) / 148));
        if (eff > best_eff + 1e-9) { best_eff = eff; best = s; }
        if (eff >= 0.9) { best = s; break; }
    }
    return best;
}

size_t workspace_size(int n_layers, int batch, int sum_nodes, int n_q_heads, int n_kv_heads, int max_pages_per_seq) {
    const int S = pick_splits(n_layers, batch, n_kv_heads, n_q_heads / n_kv_heads, max_pages_per_seq, sum_nodes);
    if (S == 1) return 16;
    return (size_t)n_layers * S * sum_nodes * n_q_heads * (kHeadDim + 2) * sizeof(float);
}

// Arguments have been validated by sage_tree_attention.
int launch(const void* q, int n_layers, int n_pages, const int32_t* page_table, int max_pages_per_seq,
           const int32_t* seq_len, const int32_t* parent, const int32_t* node_offsets, int batch, int sum_nodes,
           int n_q_heads, int n_kv_heads, float sm_scale, void* out, void* ws, int32_t* status, long long wait_cycles,
           int producer_off, int select, const CUtensorMap& kmap, const CUtensorMap& vmap, cudaStream_t stream) {
    const int G = n_q_heads / n_kv_heads;
    const int S = pick_splits(n_layers, batch, n_kv_heads, G, max_pages_per_seq, sum_nodes);
    AttnParams p{};
    p.q = (const __nv_bfloat16*)q;
    p.out = (__nv_bfloat16*)out;
    p.part_o = (float*)ws;
    p.part_ml = S > 1 ? (float*)ws + (size_t)n_layers * S * sum_nodes * n_q_heads * kHeadDim : nullptr;
    p.page_table = page_table; p.seq_len = seq_len; p.parent = parent; p.node_offsets = node_offsets;
    p.status = status;
    p.n_layers = n_layers; p.batch = batch; p.sum_nodes = sum_nodes; p.n_pages = n_pages;
    p.max_pages = max_pages_per_seq; p.Hq = n_q_heads; p.Hkv = n_kv_heads; p.G = G; p.n_splits = S;
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.wait_cycles = wait_cycles;
    p.producer_off = producer_off;
    p.select = select;
    // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SAGE_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(tree_attention_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) !=
            cudaSuccess)
            return SAGE_ERR_CUDA;
        attr_set[dev] = true;
    }
    dim3 grid(S, row_pairs_for(sum_nodes, G), n_layers * batch * n_kv_heads);
    tree_attention_split_kernel<<<grid, kAttnThreads, kSmemBytes, stream>>>(p, kmap, vmap);
    if (S > 1) {
        const size_t rows_total = (size_t)sum_nodes * n_q_heads;
        dim3 mg((unsigned)((rows_total + 7) / 8), n_layers);
        attention_split_merge_kernel<<<mg, 256, 0, stream>>>(p);
    }
    return launch_status();
}

}  // namespace split
}  // namespace sage
