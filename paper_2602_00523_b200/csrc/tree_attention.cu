// Tree-masked verification attention over a paged bf16 KV cache (Section 2.2;
// Algorithm 1, the target pass over all tree tokens; Section 3.3 Phase 2).
//
// Flash-decoding layout: the N tree nodes x G query heads that share one KV head
// form M = N*G query rows; a CTA owns a tile of those rows and one slice of the
// context (split-K), streams the slice's pages once, keeps an online softmax in
// fp32 and accumulates P.V in fp32.  Partial (m, l, O) of the slices are merged by
// a second kernel.  Key tile = one 64-token page.
#include "sage_common.cuh"

namespace sage {

constexpr int kRowsPerCta = 128;
constexpr int kAttnThreads = 256;            // 8 warps x 16 rows
constexpr int kTileBytes = kPageSize * kHeadDim * 2;   // 16 KB per K or V page tile
constexpr int kStages = 2;

struct AttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_pool;
    const __nv_bfloat16* v_pool;
    __nv_bfloat16* out;
    float* part_o;     // [layer][split][sum_nodes*Hq][128]   unnormalised
    float* part_ml;    // [layer][split][sum_nodes*Hq][2]     (m in log2 units, l)
    const int32_t* page_table;
    const int32_t* seq_len;
    const int32_t* parent;
    const int32_t* node_offsets;
    int32_t* status;
    int64_t layer_stride;
    int n_layers, batch, sum_nodes, n_pages, max_pages;
    int Hq, Hkv, G, n_splits;
    float scale_log2;  // sm_scale * log2(e)
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;   // size 0: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Tile byte offset of (key row, 16-byte chunk) with an XOR swizzle against bank conflicts.
__device__ __forceinline__ uint32_t tile_off(int key, int chunk) { return key * 256 + ((chunk ^ (key & 7)) << 4); }

__global__ void __launch_bounds__(kAttnThreads, 1) tree_attention_kernel(AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint64_t s_anc[SAGE_MAX_NODES];
    __shared__ int s_flag;
    uint8_t* sK = smem;                          // [kStages][16 KB]
    uint8_t* sV = smem + kStages * kTileBytes;   // [kStages][16 KB]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, rtile = blockIdx.y;
    const int g = blockIdx.z % p.Hkv;
    const int b = (blockIdx.z / p.Hkv) % p.batch;
    const int layer = blockIdx.z / (p.Hkv * p.batch);

    const int n0 = p.node_offsets[b];
    const int N = p.node_offsets[b + 1] - n0;
    const int L = p.seq_len[b];
    if (tid == 0) s_flag = 0;
    __syncthreads();
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
    if (rtile * kRowsPerCta >= M) return;

    // ancestor bitsets of this tree
    if (tid < SAGE_MAX_NODES) {
        uint64_t a = 0;
        if (tid < N) {
            bool bad = false;
            a = ancestor_bits(p.parent + n0, N, tid, &bad);
            if (bad) { s_flag = 1; a = 1ull << tid; }
        }
        s_anc[tid] = a;
    }
    __syncthreads();
    if (s_flag) {
        if (tid == 0) report_status(p.status, SAGE_STATUS_BAD_TREE);
        return;
    }

    const int n_tiles = (T + kPageSize - 1) / kPageSize;
    const int per_split = (n_tiles + p.n_splits - 1) / p.n_splits;
    const int t_begin = split * per_split;
    const int t_end = min(n_tiles, t_begin + per_split);

    // the two rows this thread owns inside its warp's 16-row slab
    const int r_lo = rtile * kRowsPerCta + warp * 16 + (lane >> 2);
    const int r_hi = r_lo + 8;
    const bool v_lo = r_lo < M, v_hi = r_hi < M;
    const int node_lo = v_lo ? r_lo / p.G : 0, node_hi = v_hi ? r_hi / p.G : 0;
    const int h_lo = g * p.G + (v_lo ? r_lo % p.G : 0), h_hi = g * p.G + (v_hi ? r_hi % p.G : 0);
    const size_t qrow_lo = ((size_t)layer * p.sum_nodes + n0 + node_lo) * p.Hq + h_lo;
    const size_t qrow_hi = ((size_t)layer * p.sum_nodes + n0 + node_hi) * p.Hq + h_hi;
    const uint64_t anc_lo = s_anc[node_lo], anc_hi = s_anc[node_hi];

    // Q fragments (A operand, 16 rows x 128 d): 8 k-steps x 4 registers
    uint32_t qf[8][4];
    {
        const uint32_t* qlo = reinterpret_cast<const uint32_t*>(p.q + qrow_lo * kHeadDim);
        const uint32_t* qhi = reinterpret_cast<const uint32_t*>(p.q + qrow_hi * kHeadDim);
        const int c = lane & 3;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qf[ks][0] = v_lo ? qlo[ks * 8 + c] : 0u;
            qf[ks][1] = v_hi ? qhi[ks * 8 + c] : 0u;
            qf[ks][2] = v_lo ? qlo[ks * 8 + 4 + c] : 0u;
            qf[ks][3] = v_hi ? qhi[ks * 8 + 4 + c] : 0u;
        }
    }

    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

    const __nv_bfloat16* kbase = p.k_pool + (int64_t)layer * p.layer_stride;
    const __nv_bfloat16* vbase = p.v_pool + (int64_t)layer * p.layer_stride;

    auto load_tile = [&](int t, int stage) {
        int page = p.page_table[(size_t)b * p.max_pages + t];
        if (page < 0 || page >= p.n_pages) {
            report_status(p.status, SAGE_STATUS_BAD_PAGE);
            page = 0;
        }
        const int64_t off = ((int64_t)page * p.Hkv + g) * (kPageSize * kHeadDim);
        const int valid_keys = min(kPageSize, T - t * kPageSize);
        const uint32_t dk = smem_u32(sK + stage * kTileBytes), dv = smem_u32(sV + stage * kTileBytes);
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int c = tid + it * kAttnThreads;      // 1024 chunks of 16 bytes
            const int key = c >> 4, ch = c & 15;
            const bool ok = key < valid_keys;
            cp_async_16(dk + tile_off(key, ch), kbase + off + key * kHeadDim + ch * 8, ok);
            cp_async_16(dv + tile_off(key, ch), vbase + off + key * kHeadDim + ch * 8, ok);
        }
    };

    if (t_begin < t_end) load_tile(t_begin, 0);
    cp_async_commit();

    for (int t = t_begin; t < t_end; ++t) {
        const int stage = (t - t_begin) & 1;
        if (t + 1 < t_end) load_tile(t + 1, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();

        const uint32_t kaddr = smem_u32(sK + stage * kTileBytes), vaddr = smem_u32(sV + stage * kTileBytes);
        // S = Q K^T : 16 rows x 64 keys
        float s[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                const int key = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                const int ch = ks * 2 + ((lane >> 3) & 1);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(kaddr + tile_off(key, ch), b0, b1, b2, b3);
                mma_bf16_16816(s[np * 2], qf[ks], b0, b1);
                mma_bf16_16816(s[np * 2 + 1], qf[ks], b2, b3);
            }
        }
        // scale to log2 units and mask the tree part of the tile
        const int pos0 = t * kPageSize;
        const bool need_mask = pos0 + kPageSize > L;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = s[nt][e] * p.scale_log2;
                if (need_mask) {
                    const int j = pos0 + nt * 8 + (lane & 3) * 2 + (e & 1) - L;   // tree slot, <0 = prefix
                    const uint64_t anc = (e < 2) ? anc_lo : anc_hi;
                    const bool vis = j < 0 || (j < N && ((anc >> j) & 1ull));
                    v = vis ? v : -INFINITY;
                }
                s[nt][e] = v;
            }
        }
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            mx_lo = fmaxf(mx_lo, fmaxf(s[nt][0], s[nt][1]));
            mx_hi = fmaxf(mx_hi, fmaxf(s[nt][2], s[nt][3]));
        }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
        const float base_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, base_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
        const float a_lo = exp2f(m_lo - base_lo), a_hi = exp2f(m_hi - base_hi);
        m_lo = mn_lo; m_hi = mn_hi;
        float sum_lo = 0.f, sum_hi = 0.f;
        uint32_t pf[4][4];                         // P as A fragments: 4 k-steps of 16 keys
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float p0 = exp2f(s[nt][0] - base_lo), p1 = exp2f(s[nt][1] - base_lo);
            const float p2 = exp2f(s[nt][2] - base_hi), p3 = exp2f(s[nt][3] - base_hi);
            sum_lo += p0 + p1;
            sum_hi += p2 + p3;
            pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
            pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        sum_lo += __shfl_xor_sync(0xffffffffu, sum_lo, 1);
        sum_lo += __shfl_xor_sync(0xffffffffu, sum_lo, 2);
        sum_hi += __shfl_xor_sync(0xffffffffu, sum_hi, 1);
        sum_hi += __shfl_xor_sync(0xffffffffu, sum_hi, 2);
        l_lo = l_lo * a_lo + sum_lo;
        l_hi = l_hi * a_hi + sum_hi;
#pragma unroll
        for (int i = 0; i < 16; ++i) { o[i][0] *= a_lo; o[i][1] *= a_lo; o[i][2] *= a_hi; o[i][3] *= a_hi; }
        // O += P V : k over 64 keys (4 steps), n over 128 d (16 tiles)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
            for (int np = 0; np < 8; ++np) {
                const int key = ks * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                const int ch = np * 2 + (lane >> 4);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(vaddr + tile_off(key, ch), b0, b1, b2, b3);
                mma_bf16_16816(o[np * 2], pf[ks], b0, b1);
                mma_bf16_16816(o[np * 2 + 1], pf[ks], b2, b3);
            }
        }
        __syncthreads();   // everyone is done with this stage before it is refilled
    }
    cp_async_wait<0>();

    // ---- epilogue
    const int c2 = (lane & 3) * 2;
    if (p.n_splits == 1) {
        const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
        if (v_lo) {
            uint32_t* dst = reinterpret_cast<uint32_t*>(p.out + qrow_lo * kHeadDim);
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) dst[(nt * 8 + c2) >> 1] = pack_bf16(o[nt][0] * inv_lo, o[nt][1] * inv_lo);
        }
        if (v_hi) {
            uint32_t* dst = reinterpret_cast<uint32_t*>(p.out + qrow_hi * kHeadDim);
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) dst[(nt * 8 + c2) >> 1] = pack_bf16(o[nt][2] * inv_hi, o[nt][3] * inv_hi);
        }
    } else {
        const size_t rows_total = (size_t)p.sum_nodes * p.Hq;
        const size_t slab = ((size_t)layer * p.n_splits + split) * rows_total;
        if (v_lo) {
            const size_t r = slab + (size_t)(n0 + node_lo) * p.Hq + h_lo;
            float2* dst = reinterpret_cast<float2*>(p.part_o + r * kHeadDim);
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) dst[(nt * 8 + c2) >> 1] = make_float2(o[nt][0], o[nt][1]);
            if ((lane & 3) == 0) { p.part_ml[r * 2] = m_lo; p.part_ml[r * 2 + 1] = l_lo; }
        }
        if (v_hi) {
            const size_t r = slab + (size_t)(n0 + node_hi) * p.Hq + h_hi;
            float2* dst = reinterpret_cast<float2*>(p.part_o + r * kHeadDim);
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) dst[(nt * 8 + c2) >> 1] = make_float2(o[nt][2], o[nt][3]);
            if ((lane & 3) == 0) { p.part_ml[r * 2] = m_hi; p.part_ml[r * 2 + 1] = l_hi; }
        }
    }
}

// Split-K merge: one warp per (layer, node, head) row.  Lanes first reduce (m, l) over
// the splits with shuffles, then each lane combines its four output columns.
__global__ void attention_merge_kernel(AttnParams p) {
    const int warps = blockDim.x >> 5;
    const size_t rows_total = (size_t)p.sum_nodes * p.Hq;
    const size_t row = (size_t)blockIdx.x * warps + (threadIdx.x >> 5);
    const int layer = blockIdx.y;
    const int lane = threadIdx.x & 31;
    if (row >= rows_total) return;
    const int node = (int)(row / p.Hq);
    if (node >= p.node_offsets[p.batch]) return;       // rows past the live nodes were never written
    float m = -INFINITY, l = 0.f;
    if (lane < p.n_splits) {
        const size_t r = ((size_t)layer * p.n_splits + lane) * rows_total + row;
        m = p.part_ml[r * 2];
        l = p.part_ml[r * 2 + 1];
    }
    float mx = m;
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float w = (l > 0.f) ? exp2f(m - mx) : 0.f;   // weight of this lane's split
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

static int pick_splits(int n_layers, int batch, int n_kv_heads, int G, int max_pages) {
    // enough CTAs for ~2 waves of 148 SMs, at least 4 pages per slice, at most 32 slices
    const int row_tiles = (SAGE_MAX_NODES * G + kRowsPerCta - 1) / kRowsPerCta;
    const long base = (long)n_layers * batch * n_kv_heads * row_tiles;
    long s = (2 * 148 + base - 1) / base;
    const int by_len = max_pages / 4 > 0 ? max_pages / 4 : 1;
    if (s > by_len) s = by_len;
    if (s > 32) s = 32;
    if (s < 1) s = 1;
    return (int)s;
}

}  // namespace sage

using namespace sage;

extern "C" size_t sage_tree_attention_workspace_size(int n_layers, int batch, int sum_nodes, int n_q_heads,
                                                     int n_kv_heads, int head_dim, int max_pages_per_seq) {
    if (n_layers < 1 || batch < 1 || sum_nodes < 1 || n_q_heads < 1 || n_kv_heads < 1 || max_pages_per_seq < 1) return 0;
    const int S = pick_splits(n_layers, batch, n_kv_heads, n_q_heads / n_kv_heads, max_pages_per_seq);
    if (S == 1) return 16;
    return (size_t)n_layers * S * sum_nodes * n_q_heads * (head_dim + 2) * sizeof(float);
}

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
    if ((long)n_layers * batch * n_kv_heads > 65535) return SAGE_ERR_UNSUPPORTED;
    if ((((uintptr_t)q | (uintptr_t)k_pool | (uintptr_t)v_pool | (uintptr_t)out) & 15) || (layer_stride_elems & 7))
        return SAGE_ERR_INVALID_ARG;
    if (batch == 0) return SAGE_OK;
    const int S = pick_splits(n_layers, batch, n_kv_heads, G, max_pages_per_seq);
    const size_t need = sage_tree_attention_workspace_size(n_layers, batch, sum_nodes, n_q_heads, n_kv_heads,
                                                           head_dim, max_pages_per_seq);
    if (S > 1 && (!ws || ws_bytes < need || ((uintptr_t)ws & 15))) return SAGE_ERR_WORKSPACE;
    AttnParams p{};
    p.q = (const __nv_bfloat16*)q; p.k_pool = (const __nv_bfloat16*)k_pool; p.v_pool = (const __nv_bfloat16*)v_pool;
    p.out = (__nv_bfloat16*)out;
    p.part_o = (float*)ws;
    p.part_ml = S > 1 ? (float*)ws + (size_t)n_layers * S * sum_nodes * n_q_heads * kHeadDim : nullptr;
    p.page_table = page_table; p.seq_len = seq_len; p.parent = parent; p.node_offsets = node_offsets;
    p.status = status; p.layer_stride = layer_stride_elems;
    p.n_layers = n_layers; p.batch = batch; p.sum_nodes = sum_nodes; p.n_pages = n_pages;
    p.max_pages = max_pages_per_seq; p.Hq = n_q_heads; p.Hkv = n_kv_heads; p.G = G; p.n_splits = S;
    p.scale_log2 = sm_scale * 1.4426950408889634f;

    static bool attr_set = false;
    const int smem = 2 * kStages * kTileBytes;
    if (!attr_set) {
        if (cudaFuncSetAttribute(tree_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return SAGE_ERR_CUDA;
        attr_set = true;
    }
    const int row_tiles = (SAGE_MAX_NODES * G + kRowsPerCta - 1) / kRowsPerCta;
    dim3 grid(S, row_tiles, n_layers * batch * n_kv_heads);
    tree_attention_kernel<<<grid, kAttnThreads, smem, as_stream(stream)>>>(p);
    if (S > 1) {
        const size_t rows_total = (size_t)sum_nodes * n_q_heads;
        dim3 mg((unsigned)((rows_total + 7) / 8), n_layers);
        attention_merge_kernel<<<mg, 256, 0, as_stream(stream)>>>(p);
    }
    return launch_status();
}
