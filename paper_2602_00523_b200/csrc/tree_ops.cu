// Tree-side kernels of the SAGE decode round: template selection, ancestor
// bitsets, draft-token expansion, greedy acceptance and KV compaction.
// All of them are latency-bound (a few hundred bytes to a few MB per round).
#include "sage_common.cuh"

namespace sage {

// ---------------------------------------------------------------------------
// alpha -> template (Eq. 10 / Eq. 11, Section 3.2) + optional hand-over of the
// chosen templates' parent/rank arrays for the next round.
// ---------------------------------------------------------------------------
struct SelectParams {
    const float* alpha;
    const int32_t* alpha_row;
    int batch;
    sage_tree_policy pol;
    int32_t* template_id;
    float* depth_cont;
    float* width_cont;
    const int32_t* bank_parent;
    const int32_t* bank_rank;
    const int32_t* bank_n_nodes;
    int32_t* next_parent;
    int32_t* next_rank;
    int32_t* next_node_offsets;
    int32_t* status;
};

__device__ __forceinline__ int pick_template(const SelectParams& p, int b, float* a_out) {
    const int row = p.alpha_row ? p.alpha_row[b] : b;
    const float a = p.alpha[row];
    int t = 0;
    for (int j = 0; j + 1 < p.pol.n_templates; ++j) t += (a < p.pol.alpha_thresholds[j]) ? 1 : 0;
    *a_out = a;
    return t;
}

__global__ void select_tree_kernel(SelectParams p) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= p.batch) return;
    float a;
    const int t = pick_template(p, b, &a);
    p.template_id[b] = t;
    if (p.depth_cont) p.depth_cont[b] = fmaf(a, p.pol.d_max - p.pol.d_min, p.pol.d_min);
    if (p.width_cont) p.width_cont[b] = fmaf(1.0f - a, p.pol.w_max - p.pol.w_min, p.pol.w_min);
}

// One block: offsets are a running sum over the batch, then every tree is copied.
__global__ void handover_trees_kernel(SelectParams p) {
    __shared__ int s_bad;
    if (threadIdx.x == 0) {
        int off = 0, bad = 0;
        for (int b = 0; b < p.batch; ++b) {
            p.next_node_offsets[b] = off;
            int n = p.bank_n_nodes[p.template_id[b]];
            if (n < 1 || n > SAGE_MAX_NODES) { bad = 1; n = 1; }
            off += n;
        }
        p.next_node_offsets[p.batch] = off;
        s_bad = bad;
        if (bad) report_status(p.status, SAGE_STATUS_BAD_TREE);
    }
    __syncthreads();
    if (s_bad) return;
    for (int b = 0; b < p.batch; ++b) {
        const int t = p.template_id[b];
        const int n = p.bank_n_nodes[t];
        const int off = p.next_node_offsets[b];
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            p.next_parent[off + i] = p.bank_parent[t * SAGE_MAX_NODES + i];
            p.next_rank[off + i] = p.bank_rank[t * SAGE_MAX_NODES + i];
        }
    }
}

// ---------------------------------------------------------------------------
// Ancestor bitsets (Section 2.2; Algorithm 1 TreeAttnMask)
// ---------------------------------------------------------------------------
__global__ void ancestor_mask_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ node_offsets,
                                     uint64_t* __restrict__ anc, int32_t* status) {
    const int b = blockIdx.x;
    const int n0 = node_offsets[b];
    const int n = node_offsets[b + 1] - n0;
    if (n < 1 || n > SAGE_MAX_NODES) {
        if (threadIdx.x == 0) report_status(status, SAGE_STATUS_BAD_TREE);
        return;
    }
    const int i = threadIdx.x;
    if (i >= n) return;
    bool bad = false;
    const uint64_t a = ancestor_bits(parent + n0, n, i, &bad);
    if (bad) report_status(status, SAGE_STATUS_BAD_TREE);
    anc[n0 + i] = bad ? (1ull << i) : a;
}

// ---------------------------------------------------------------------------
// Greedy acceptance, one warp per tree (Section 2.2, Eq. 5; Section 3.3 Phase 2).
// Node i is accepted iff every non-root node on its root path matches the
// target's argmax at its parent.  With anc(i) as a bitset and `match` the bitset
// of matching nodes this is (anc(i) & ~match) == 0.  Because parent < child, a
// root path read in increasing node index is the path itself, so "longest, then
// lexicographically smallest" is the maximum of (depth, bit-reversed anc(i)).
// ---------------------------------------------------------------------------
__global__ void accept_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ draft_token,
                              const int32_t* __restrict__ target_argmax, const int32_t* __restrict__ node_offsets,
                              int batch, int max_path, int32_t* __restrict__ path, int32_t* __restrict__ path_len,
                              int32_t* __restrict__ bonus_token, int32_t* status) {
    const int warps_per_block = blockDim.x >> 5;
    const int b = blockIdx.x * warps_per_block + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= batch) return;
    const int n0 = node_offsets[b];
    const int n = node_offsets[b + 1] - n0;
    int32_t* my_path = path + (size_t)b * max_path;
    bool bad_tree = (n < 1 || n > SAGE_MAX_NODES);
    uint64_t anc[2] = {0, 0};
    bool match[2] = {false, false};
    if (!bad_tree) {
        for (int u = 0; u < 2; ++u) {
            const int i = lane + 32 * u;
            if (i < n) {
                bool bad = false;
                anc[u] = ancestor_bits(parent + n0, n, i, &bad);
                bad_tree |= bad;
                if (!bad) match[u] = (i == 0) || (draft_token[n0 + i] == target_argmax[n0 + parent[n0 + i]]);
            }
        }
    }
    bad_tree = __any_sync(0xffffffffu, bad_tree);
    if (bad_tree) {
        if (lane == 0) {
            report_status(status, SAGE_STATUS_BAD_TREE);
            path_len[b] = 0;
            bonus_token[b] = -1;
        }
        for (int j = lane; j < max_path; j += 32) my_path[j] = -1;
        return;
    }
    const uint64_t match_bits = (uint64_t)__ballot_sync(0xffffffffu, match[0]) |
                                ((uint64_t)__ballot_sync(0xffffffffu, match[1]) << 32);
    // best key over accepted nodes: depth first, then bit-reversed ancestor set
    int best_depth = -1;
    uint64_t best_rev = 0, best_anc = 0;
    for (int u = 0; u < 2; ++u) {
        const int i = lane + 32 * u;
        if (i < n && (anc[u] & ~match_bits) == 0) {
            const int len = __popcll(anc[u]);   // nodes on the path = depth + 1
            if (len <= max_path) {
                const uint64_t rev = __brevll(anc[u]);
                if (len > best_depth || (len == best_depth && rev > best_rev)) {
                    best_depth = len; best_rev = rev; best_anc = anc[u];
                }
            }
        }
    }
    for (int off = 16; off > 0; off >>= 1) {
        const int od = __shfl_xor_sync(0xffffffffu, best_depth, off);
        const uint64_t orv = __shfl_xor_sync(0xffffffffu, best_rev, off);
        const uint64_t oan = __shfl_xor_sync(0xffffffffu, best_anc, off);
        if (od > best_depth || (od == best_depth && orv > best_rev)) {
            best_depth = od; best_rev = orv; best_anc = oan;
        }
    }
    // best_anc holds the accepted path (the root alone is always accepted: len 1 <= max_path)
    const int len = __popcll(best_anc);
    for (int j = lane; j < max_path; j += 32) {
        int node = -1;
        if (j < len) {
            uint64_t m = best_anc;
            for (int s = 0; s < j; ++s) m &= m - 1;      // drop the j lowest set bits
            node = __ffsll((long long)m) - 1;
        }
        my_path[j] = node;
    }
    if (lane == 0) {
        path_len[b] = len;
        bonus_token[b] = target_argmax[n0 + (63 - __clzll((long long)best_anc))];
    }
}

// ---------------------------------------------------------------------------
// KV compaction (Algorithm 1 cache update).  One block per (sequence, layer):
// thread = one 16-byte chunk of one (K or V, kv head) row.  Destinations L+j
// never lie above their sources L+path[j] (path[j] >= j because parent < child),
// and sources of later j lie above every earlier destination, so walking j
// upwards with "read a batch, then write it" needs no barrier.
// ---------------------------------------------------------------------------
struct CompactParams {
    __nv_bfloat16* k_pool;
    __nv_bfloat16* v_pool;
    int64_t layer_stride;
    int n_layers, n_pages, max_pages, batch, max_path, n_kv_heads;
    const int32_t* page_table;
    const int32_t* seq_len;
    const int32_t* path;
    const int32_t* path_len;
    int32_t* status;
};

// Checks one sequence's accepted path and, when `src` / `dst` are given, turns it into element
// offsets of the (page, head 0, slot) rows to move (-1 = row already in place).  Returns the
// number of path entries, or 0 with *code set when the path or a page id is not valid: such a
// sequence is left exactly as it is (nothing moves, its length does not advance).
__device__ int plan_compaction(const CompactParams& p, int b, int64_t* src, int64_t* dst, int* code) {
    const int L = p.seq_len[b];
    int plen = p.path_len[b];
    bool bad_path = (plen < 0 || plen > p.max_path || plen > SAGE_MAX_NODES || L < 0);
    bool bad_page = false;
    if (bad_path) plen = 0;
    int prev = -1;
    for (int j = 0; j < plen; ++j) {
        const int node = p.path[(size_t)b * p.max_path + j];
        int64_t so = -1, dofs = -1;
        if (node <= prev || node < j || node >= SAGE_MAX_NODES || (j == 0 && node != 0)) {
            bad_path = true;                       // a root path starts at 0 and visits increasing indices
        } else if (node != j) {
            const int s_pos = L + node, d_pos = L + j;
            if (s_pos / kPageSize >= p.max_pages) {
                bad_page = true;
            } else {
                const int sp = p.page_table[(size_t)b * p.max_pages + s_pos / kPageSize];
                const int dp = p.page_table[(size_t)b * p.max_pages + d_pos / kPageSize];
                if (sp < 0 || sp >= p.n_pages || dp < 0 || dp >= p.n_pages) {
                    bad_page = true;
                } else {
                    so = ((int64_t)sp * p.n_kv_heads * kPageSize + s_pos % kPageSize) * kHeadDim;
                    dofs = ((int64_t)dp * p.n_kv_heads * kPageSize + d_pos % kPageSize) * kHeadDim;
                }
            }
        }
        prev = node;
        if (src) { src[j] = so; dst[j] = dofs; }
    }
    *code = bad_path ? SAGE_STATUS_BAD_PATH : (bad_page ? SAGE_STATUS_BAD_PAGE : 0);
    return *code ? 0 : plen;
}

__global__ void __launch_bounds__(256) compact_kv_kernel(CompactParams p) {
    __shared__ int64_t s_src[SAGE_MAX_NODES];   // element offset of (page, head 0, slot) rows, -1 = skip
    __shared__ int64_t s_dst[SAGE_MAX_NODES];
    __shared__ int s_len;
    const int b = blockIdx.x;
    const int layer = blockIdx.y;
    if (threadIdx.x == 0) {
        int code = 0;
        s_len = plan_compaction(p, b, s_src, s_dst, &code);
        if (code) report_status(p.status, code);
    }
    __syncthreads();
    const int plen = s_len;
    const int cols = p.n_kv_heads * 16;          // 16-byte chunks per token row across heads
    for (int c = threadIdx.x; c < 2 * cols; c += blockDim.x) {
        __nv_bfloat16* pool = (c < cols ? p.k_pool : p.v_pool) + (int64_t)layer * p.layer_stride;
        const int cc = c % cols;
        const int64_t col = (int64_t)(cc / 16) * kPageSize * kHeadDim + (cc % 16) * 8;
        for (int j0 = 0; j0 < plen; j0 += 8) {
            uint4 r[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u;
                if (j < plen && s_src[j] >= 0) r[u] = *reinterpret_cast<const uint4*>(pool + s_src[j] + col);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u;
                if (j < plen && s_src[j] >= 0) *reinterpret_cast<uint4*>(pool + s_dst[j] + col) = r[u];
            }
        }
    }
}

// Runs after compact_kv_kernel (same stream): a sequence's length advances only when its path
// passed the same checks, i.e. only when its rows were actually moved.
__global__ void advance_seq_len_kernel(CompactParams p, int32_t* seq_len) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= p.batch) return;
    int code = 0;
    const int plen = plan_compaction(p, b, nullptr, nullptr, &code);
    if (!code) seq_len[b] += plen;
}

// ---------------------------------------------------------------------------
// Dynamic tree construction, one level per launch (Section 3.2: hierarchical width
// decay, Eq. 12, and "Dynamic Tree Construction").  One block per sequence, one
// thread per frontier node.  A child of rank r of frontier node u joins the tree iff
// r < W_l and exp(cum_logprob) > theta_l; both tests only ever cut a suffix of the
// (descending) candidate row, so each node contributes a prefix of its ranks, and the
// children are laid out in breadth-first order by a prefix sum.  Decisions are taken
// in fp64 on the fp32 inputs; cumulative log-probabilities are fp32 sums.
// ---------------------------------------------------------------------------
struct GrowParams {
    const int32_t* topk_idx;
    const float* topk_logprob;
    int k;
    const float* alpha;
    const int32_t* alpha_row;
    sage_tree_policy pol;
    int n_max;
    int32_t *parent, *rank, *depth, *token;
    float* cum_logprob;
    int32_t *n_nodes, *frontier_begin;
    const float* d_max_seq;
    int32_t* status;
};

__global__ void __launch_bounds__(SAGE_MAX_NODES) grow_tree_kernel(GrowParams p) {
    __shared__ int s_count[SAGE_MAX_NODES];
    const int b = blockIdx.x, tid = threadIdx.x;
    const int base = b * SAGE_MAX_NODES;
    const int n = p.n_nodes[b], fb = p.frontier_begin[b];
    if (n < 1 || n > p.n_max || fb < 0 || fb > n) {
        if (tid == 0) report_status(p.status, SAGE_STATUS_BAD_TREE);
        return;
    }
    if (fb == n) return;                                   // nothing left to expand
    const int level = p.depth[base + fb] + 1;
    const double a = (double)p.alpha[p.alpha_row ? p.alpha_row[b] : b];
    // explicit roundings: no fused multiply-add, so that a host check in plain fp64 sees the same D and W
    const double d_max = p.d_max_seq ? (double)p.d_max_seq[b] : (double)p.pol.d_max;
    const double D = __dadd_rn((double)p.pol.d_min, __dmul_rn(a, d_max - (double)p.pol.d_min));
    const double W = __dadd_rn((double)p.pol.w_min, __dmul_rn(1.0 - a, (double)p.pol.w_max - (double)p.pol.w_min));
    if ((double)level > D) {                               // the tree has reached its depth
        if (tid == 0) p.frontier_begin[b] = n;
        return;
    }
    const double theta = 0.1 * (double)level / D;
    const int node = fb + tid;
    int count = 0;
    float cum_u = 0.f;
    if (node < n) {
        cum_u = p.cum_logprob[base + node];
        const double p_parent = exp((double)cum_u);
        const double w_l = (level == 1) ? W : W / (double)level * (0.5 + p_parent);
        const float* lp = p.topk_logprob + (size_t)(base + node) * p.k;
        for (int r = 0; r < p.k; ++r) {
            if (!((double)r < w_l)) break;
            const float c = __fadd_rn(cum_u, lp[r]);
            if (!(exp((double)c) > theta)) break;
            ++count;
        }
    }
    s_count[tid] = count;
    __syncthreads();
    int before = 0, total = 0;
    for (int i = 0; i < SAGE_MAX_NODES; ++i) {
        const int c = s_count[i];
        if (i < tid) before += c;
        total += c;
    }
    if (node < n) {
        const float* lp = p.topk_logprob + (size_t)(base + node) * p.k;
        const int32_t* ix = p.topk_idx + (size_t)(base + node) * p.k;
        for (int r = 0; r < count; ++r) {
            const int pos = n + before + r;
            if (pos >= p.n_max) break;                     // node budget: breadth-first prefix
            p.parent[base + pos] = node;
            p.rank[base + pos] = r;
            p.depth[base + pos] = level;
            p.token[base + pos] = ix[r];
            p.cum_logprob[base + pos] = __fadd_rn(cum_u, lp[r]);
        }
    }
    if (tid == 0) {
        p.n_nodes[b] = min(n + total, p.n_max);
        p.frontier_begin[b] = n;
    }
}

// ---------------------------------------------------------------------------
// Adaptive history tracking (Section 3.3; window 10, thresholds 2 and 3 in Section 5.1).
// One thread per sequence: push tau = path_len - 1 into the sequence's ring of recent
// acceptance lengths; once `min_samples` values are there, their mean below `lower`
// lowers the sequence's maximum depth by `step`, above `upper` raises it, clamped to
// [d_lo, d_hi].  The mean is an exact integer sum divided in fp64.
// ---------------------------------------------------------------------------
__global__ void update_history_kernel(const int32_t* __restrict__ path_len, int batch, sage_history_policy pol,
                                      int32_t* __restrict__ window_buf, int32_t* __restrict__ count,
                                      float* __restrict__ d_max, int32_t* status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int pl = path_len[b];
    const int c = count[b];
    if (pl < 1 || c < 0) {                          // the root is always accepted: path_len >= 1
        report_status(status, SAGE_STATUS_BAD_PATH);
        return;
    }
    int32_t* ring = window_buf + (size_t)b * pol.window;
    ring[c % pol.window] = pl - 1;
    count[b] = c + 1;
    const int n = min(c + 1, pol.window);
    if (n < pol.min_samples) return;
    long long sum = 0;
    for (int i = 0; i < n; ++i) sum += ring[i];
    const double mean = (double)sum / (double)n;
    float d = d_max[b];
    if (mean < (double)pol.lower) d = fmaxf(pol.d_lo, d - pol.step);
    else if (mean > (double)pol.upper) d = fminf(pol.d_hi, d + pol.step);
    d_max[b] = d;
}

}  // namespace sage

using namespace sage;

extern "C" int sage_select_tree(const float* alpha, const int32_t* alpha_row, int batch,
                                const sage_tree_policy* policy, int32_t* template_id, float* depth_cont,
                                float* width_cont, const int32_t* bank_parent, const int32_t* bank_rank,
                                const int32_t* bank_n_nodes, int32_t* next_parent, int32_t* next_rank,
                                int32_t* next_node_offsets, int32_t* status, void* stream) {
    if (!alpha || !policy || !template_id || batch < 0) return SAGE_ERR_INVALID_ARG;
    if (policy->n_templates < 1 || policy->n_templates > SAGE_MAX_TEMPLATES) return SAGE_ERR_INVALID_ARG;
    for (int j = 0; j + 2 < policy->n_templates; ++j)
        if (!(policy->alpha_thresholds[j] >= policy->alpha_thresholds[j + 1])) return SAGE_ERR_INVALID_ARG;
    const bool handover = next_parent != nullptr;
    if (handover && (!bank_parent || !bank_rank || !bank_n_nodes || !next_rank || !next_node_offsets))
        return SAGE_ERR_INVALID_ARG;
    if (batch == 0) return SAGE_OK;
    SelectParams p{alpha, alpha_row, batch, *policy, template_id, depth_cont, width_cont, bank_parent,
                   bank_rank, bank_n_nodes, next_parent, next_rank, next_node_offsets, status};
    select_tree_kernel<<<(batch + 127) / 128, 128, 0, as_stream(stream)>>>(p);
    if (handover) handover_trees_kernel<<<1, 256, 0, as_stream(stream)>>>(p);
    return launch_status();
}

extern "C" int sage_build_ancestor_mask(const int32_t* parent, const int32_t* node_offsets, int batch,
                                        uint64_t* anc, int32_t* status, void* stream) {
    if (!parent || !node_offsets || !anc || batch < 0) return SAGE_ERR_INVALID_ARG;
    if (batch == 0) return SAGE_OK;
    ancestor_mask_kernel<<<batch, SAGE_MAX_NODES, 0, as_stream(stream)>>>(parent, node_offsets, anc, status);
    return launch_status();
}

extern "C" int sage_accept(const int32_t* parent, const int32_t* draft_token, const int32_t* target_argmax,
                           const int32_t* node_offsets, int batch, int max_path, int32_t* path,
                           int32_t* path_len, int32_t* bonus_token, int32_t* status, void* stream) {
    if (!parent || !draft_token || !target_argmax || !node_offsets || !path || !path_len || !bonus_token)
        return SAGE_ERR_INVALID_ARG;
    if (batch < 0 || max_path < 1) return SAGE_ERR_INVALID_ARG;
    if (batch == 0) return SAGE_OK;
    const int wpb = 4;
    accept_kernel<<<(batch + wpb - 1) / wpb, wpb * 32, 0, as_stream(stream)>>>(
        parent, draft_token, target_argmax, node_offsets, batch, max_path, path, path_len, bonus_token, status);
    return launch_status();
}

extern "C" int sage_compact_kv(void* k_pool, void* v_pool, int64_t layer_stride_elems, int n_layers, int n_pages,
                               const int32_t* page_table, int max_pages_per_seq, int32_t* seq_len,
                               const int32_t* path, const int32_t* path_len, int batch, int max_path,
                               int n_kv_heads, int head_dim, int page_size, int32_t* status, void* stream) {
    if (!k_pool || !v_pool || !page_table || !seq_len || !path || !path_len) return SAGE_ERR_INVALID_ARG;
    if (batch < 0 || n_layers < 1 || n_pages < 1 || max_pages_per_seq < 1 || max_path < 1 || n_kv_heads < 1 ||
        layer_stride_elems < 0)
        return SAGE_ERR_INVALID_ARG;
    if (head_dim != kHeadDim || page_size != kPageSize || n_layers > 65535) return SAGE_ERR_UNSUPPORTED;
    if (((uintptr_t)k_pool | (uintptr_t)v_pool) & 15 || (layer_stride_elems & 7)) return SAGE_ERR_INVALID_ARG;
    if (batch == 0) return SAGE_OK;
    CompactParams p{(__nv_bfloat16*)k_pool, (__nv_bfloat16*)v_pool, layer_stride_elems, n_layers, n_pages,
                    max_pages_per_seq, batch, max_path, n_kv_heads, page_table, seq_len, path, path_len, status};
    compact_kv_kernel<<<dim3(batch, n_layers), 256, 0, as_stream(stream)>>>(p);
    advance_seq_len_kernel<<<(batch + 127) / 128, 128, 0, as_stream(stream)>>>(p, seq_len);
    return launch_status();
}

extern "C" int sage_grow_tree(const int32_t* topk_idx, const float* topk_logprob, int k, const float* alpha,
                              const int32_t* alpha_row, int batch, const sage_tree_policy* policy, int n_max,
                              int32_t* parent, int32_t* rank, int32_t* depth, int32_t* token, float* cum_logprob,
                              int32_t* n_nodes, int32_t* frontier_begin, const float* d_max_seq, int32_t* status,
                              void* stream) {
    if (!topk_idx || !topk_logprob || !alpha || !policy || !parent || !rank || !depth || !token || !cum_logprob ||
        !n_nodes || !frontier_begin)
        return SAGE_ERR_INVALID_ARG;
    if (batch < 0 || k < 1 || n_max < 1) return SAGE_ERR_INVALID_ARG;
    if (k > SAGE_MAX_TOPK || n_max > SAGE_MAX_NODES) return SAGE_ERR_UNSUPPORTED;
    if (!(policy->d_max >= policy->d_min) || !(policy->d_min > 0.f) || !(policy->w_max >= policy->w_min) ||
        !(policy->w_min > 0.f))
        return SAGE_ERR_INVALID_ARG;
    if (batch == 0) return SAGE_OK;
    GrowParams p{topk_idx, topk_logprob, k, alpha, alpha_row, *policy, n_max, parent, rank, depth, token,
                 cum_logprob, n_nodes, frontier_begin, d_max_seq, status};
    grow_tree_kernel<<<batch, SAGE_MAX_NODES, 0, as_stream(stream)>>>(p);
    return launch_status();
}

extern "C" int sage_update_history(const int32_t* path_len, int batch, const sage_history_policy* policy,
                                   int32_t* window_buf, int32_t* count, float* d_max, int32_t* status,
                                   void* stream) {
    if (!path_len || !policy || !window_buf || !count || !d_max || batch < 0) return SAGE_ERR_INVALID_ARG;
    if (policy->window < 1 || policy->min_samples < 1 || policy->min_samples > policy->window ||
        !(policy->upper >= policy->lower) || !(policy->d_hi >= policy->d_lo) || !(policy->step >= 0.f))
        return SAGE_ERR_INVALID_ARG;
    if (policy->window > 1024) return SAGE_ERR_UNSUPPORTED;
    if (batch == 0) return SAGE_OK;
    update_history_kernel<<<(batch + 127) / 128, 128, 0, as_stream(stream)>>>(path_len, batch, *policy, window_buf,
                                                                              count, d_max, status);
    return launch_status();
}

extern "C" const char* sage_status_string(int code) {
    switch (code) {
        case SAGE_OK: return "ok";
        case SAGE_ERR_INVALID_ARG: return "invalid argument";
        case SAGE_ERR_UNSUPPORTED: return "outside the supported envelope";
        case SAGE_ERR_WORKSPACE: return "workspace missing or too small";
        case SAGE_ERR_CUDA: return "CUDA call failed";
        case SAGE_ERR_TOO_LARGE: return "problem needs more scratch than the library's built-in array holds";
        case SAGE_STATUS_BAD_TREE: return "device: parent array or node count violates the tree rules";
        case SAGE_STATUS_BAD_PAGE: return "device: page id out of range or sequence longer than its page table";
        case SAGE_STATUS_TIMEOUT: return "device: bounded wait expired";
        case SAGE_STATUS_BAD_PATH: return "device: accepted path is not a valid root path";
        default: return "unknown status";
    }
}
