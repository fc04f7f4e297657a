/*
 * sage.h -- C ABI of the SAGE decode-round hot path on one NVIDIA B200 (sm_100a).
 *
 * SAGE (entropy-guided adaptive speculative decoding for vision-language
 * models) runs, per decode round: tree drafting with top-k expansion, one
 * tree-masked verification pass of the target model, greedy acceptance of the
 * longest matching path, a KV-cache update, and an entropy-driven choice of the
 * next tree's depth and width (Algorithm 1, Section 3.3).  This library holds
 * the data-parallel kernels of that round.
 *
 * Conventions for every entry point
 *  - Returns SAGE_OK (0) or a SAGE_ERR_* code.  Argument errors are detected on
 *    the host before anything is enqueued.
 *  - All pointers are DEVICE pointers owned by the caller unless the comment
 *    says "host".  The library never allocates or frees device memory and
 *    never synchronises: work is enqueued on `stream` (a cudaStream_t passed as
 *    void*; NULL = the legacy default stream).  Scratch memory comes from the
 *    caller (`ws`, `ws_bytes`; sizes from the *_workspace_size queries).
 *  - `status` (int32_t[1], device, may be NULL) receives the first data-dependent
 *    error a kernel meets (SAGE_STATUS_*); kernels then return early and never
 *    trap.  The caller zeroes it and reads it back when it wants to.
 *  - Inputs are never modified, except by sage_compact_kv (pools, seq_len).
 *  - Results are deterministic run to run.
 *  - Trees: node_offsets[batch+1] delimits each sequence's nodes; within a tree
 *    node 0 is the root (the last committed token, parent = -1) and every other
 *    node i has 0 <= parent[i] < i.  At most 64 nodes per tree (N_max,
 *    Section 5.1 "Implementation details").
 *  - Paged KV cache: pools are bf16 [n_layers][n_pages][n_kv_heads][page_size][head_dim]
 *    with `layer_stride_elems` elements between layers; logical position t of
 *    sequence b lives in page page_table[b*max_pages_per_seq + t/page_size], slot
 *    t%page_size.  seq_len[b] = prefix length L_b; the K/V of the N_b tree nodes
 *    sit at logical positions L_b .. L_b+N_b-1 of the same cache.
 *  Supported envelope (else SAGE_ERR_UNSUPPORTED): head_dim = 128, page_size = 64,
 *  n_q_heads / n_kv_heads in {1,2,4,8}, k <= 16, k_entropy <= 16, finite logits.
 */
#ifndef SAGE_H_
#define SAGE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SAGE_OK               0
#define SAGE_ERR_INVALID_ARG  1   /* null pointer, negative size, bad combination      */
#define SAGE_ERR_UNSUPPORTED  2   /* outside the supported envelope                     */
#define SAGE_ERR_WORKSPACE    3   /* ws == NULL or ws_bytes too small                   */
#define SAGE_ERR_CUDA         4   /* a CUDA runtime / driver call failed                */
#define SAGE_ERR_TOO_LARGE    5   /* problem needs more scratch than the built-in array */

/* values written to the device status word (first error wins) */
#define SAGE_STATUS_BAD_TREE  101 /* parent array / node count violates the tree rules  */
#define SAGE_STATUS_BAD_PAGE  102 /* page id outside [0, n_pages) or sequence too long  */
#define SAGE_STATUS_TIMEOUT   103 /* a bounded on-device wait expired                   */
#define SAGE_STATUS_BAD_PATH  104 /* path entry outside the tree / path_len out of range*/

#define SAGE_MAX_NODES      64
#define SAGE_MAX_TOPK       16
#define SAGE_MAX_TEMPLATES  8

/* Tree policy (host struct).  Depth / width follow Eq. 10 and Eq. 11 of
 * Section 3.2: D = d_min + alpha (d_max - d_min), W = w_min + (1 - alpha)(w_max - w_min).
 * The paper does not say how the real-valued (D, W) become a concrete tree; here
 * the caller registers n_templates tree templates, ordered from the deepest /
 * narrowest to the shallowest / widest, and n_templates-1 descending alpha
 * thresholds: template_id = number of thresholds strictly greater than alpha. */
typedef struct sage_tree_policy {
    int   n_templates;                          /* 1 .. SAGE_MAX_TEMPLATES              */
    float alpha_thresholds[SAGE_MAX_TEMPLATES]; /* first n_templates-1 used, descending */
    float d_min, d_max, w_min, w_max;           /* paper: 3, 8, 2, 10                   */
} sage_tree_policy;

/* Fused softmax entropy + top-k over vocabulary-sized rows.
 * Computes, for each of `rows` fp32 logits rows (row r starts at logits + r*row_stride;
 * row_stride % 4 == 0 and logits 16-byte aligned):
 *   - the k largest logits, ordered by value descending, ties to the lowest index,
 *     -0 == +0 (Top_k of Eq. 4, Section 2.2): topk_idx[r*k + j], topk_logprob = x - logsumexp;
 *   - lse[r] = log sum exp and entropy_full[r] = Shannon entropy (nats) of softmax(row);
 *   - the entropy of the top-k_entropy probabilities renormalised to sum 1 (Eq. 7, Eq. 8,
 *     Section 3.1) in entropy_topk[r], and alpha[r] = 1 - H / ln(k_entropy) clamped to
 *     [0,1] (Eq. 9); alpha = 1 when k_entropy == 1.
 * Any of entropy_full / entropy_topk / alpha / lse / topk_logprob may be NULL.
 * Optional expansion (Section 2.2 "Tree-based Drafting", Section 3.2 "Dynamic Tree
 * Construction"): when draft_token != NULL, logits row r belongs to global node r and
 *   draft_token[i] = topk_idx[(n0 + parent[i])*k + rank[i]]  for non-root nodes,
 *   draft_token[n0] = root_token[b],   n0 = node_offsets[b];
 * then parent, rank, node_offsets, root_token must be non-NULL and rank[i] < k.
 * ws: sage_expand_topk_workspace_size(rows, vocab) bytes. */
int sage_expand_topk(const float *logits, int rows, int vocab, int64_t row_stride,
                     int k, int k_entropy,
                     int32_t *topk_idx, float *topk_logprob,
                     float *entropy_full, float *entropy_topk, float *alpha, float *lse,
                     const int32_t *parent, const int32_t *rank, const int32_t *node_offsets,
                     int batch, const int32_t *root_token, int32_t *draft_token,
                     void *ws, size_t ws_bytes, int32_t *status, void *stream);
size_t sage_expand_topk_workspace_size(int rows, int vocab);

/* sage_expand_topk for callers that cannot provide scratch memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, not another operation.)
 * Who needs it: code that runs where no device allocation is possible -- a plug-in that is
 * handed only its input and output buffers by a serving engine whose own pool already owns
 * all of the GPU's memory, or a decode loop that must not call cudaMalloc because that call
 * synchronises the whole device.  Such a caller has nowhere to get `ws` from.
 * Same arguments, results and error codes as sage_expand_topk, minus ws / ws_bytes: the
 * scratch is a fixed array of SAGE_STATIC_SCRATCH_BYTES bytes inside the library, present on
 * every GPU that loads the library, for the life of the process.  The call performs no
 * allocation of any kind.
 *  - Limit: sage_expand_topk_workspace_size(rows, vocab) must not exceed
 *    SAGE_STATIC_SCRATCH_BYTES (60 rows x 152064 need about 90 KB; several thousand rows
 *    fit); otherwise SAGE_ERR_TOO_LARGE is returned and nothing is enqueued.
 *  - The first call on each device looks up the array's device address (a runtime query,
 *    done with that device current, which also loads the library's kernels there).  Make
 *    that first call before starting any stream capture on that device.
 *  - All calls on one device use the same array, and it keeps whatever the previous call
 *    left; the kernels overwrite every slot they later read, so no clearing is needed.  Two
 *    calls that may run at the same time on one GPU (different streams, or different host
 *    threads) race on the array and give wrong results: keep them ordered on one stream. */
#define SAGE_STATIC_SCRATCH_BYTES (1 << 20)
int sage_expand_topk_static(const float *logits, int rows, int vocab, int64_t row_stride,
                            int k, int k_entropy,
                            int32_t *topk_idx, float *topk_logprob,
                            float *entropy_full, float *entropy_topk, float *alpha, float *lse,
                            const int32_t *parent, const int32_t *rank, const int32_t *node_offsets,
                            int batch, const int32_t *root_token, int32_t *draft_token,
                            int32_t *status, void *stream);

/* Confidence -> tree template (Eq. 10, Eq. 11; Algorithm 1 "Phase 3: Dynamic Tree
 * Update").  For sequence b the confidence is alpha[alpha_row ? alpha_row[b] : b]
 * (which row of a tree supplies the distribution is the caller's choice).  Writes
 * template_id[b] and the unrounded D(alpha), W(alpha) (fp32, one fused multiply-add
 * each; either may be NULL).  `policy` is a host pointer, read during the call.
 * Optional device-side tree hand-over for the NEXT round (the look-ahead of Section 3.2
 * "Temporal Correlation Exploitation"), so that no host round trip is needed: when
 * next_parent != NULL, bank_parent / bank_rank hold the templates' arrays
 * ([n_templates][SAGE_MAX_NODES] int32) and bank_n_nodes[n_templates] their sizes; the
 * call writes next_node_offsets[batch+1] (prefix sums of the chosen sizes) and the
 * chosen templates' parent / rank arrays packed at those offsets
 * (capacity batch*SAGE_MAX_NODES). */
int sage_select_tree(const float *alpha, const int32_t *alpha_row, int batch,
                     const sage_tree_policy *policy,
                     int32_t *template_id, float *depth_cont, float *width_cont,
                     const int32_t *bank_parent, const int32_t *bank_rank, const int32_t *bank_n_nodes,
                     int32_t *next_parent, int32_t *next_rank, int32_t *next_node_offsets,
                     int32_t *status, void *stream);

/* Dynamic tree construction, one level per call (Section 3.2: "Hierarchical Width Decay", Eq. 12,
 * and "Dynamic Tree Construction"; Algorithm 1, the tree update of phase 3).  Every sequence b owns
 * SAGE_MAX_NODES node slots: slot b*SAGE_MAX_NODES + i holds node i (parent, rank among its parent's
 * candidates, depth, token, cum_logprob = log of the cumulative path probability).  Nodes
 * frontier_begin[b] .. n_nodes[b]-1 are the deepest level so far; row b*SAGE_MAX_NODES + i of
 * topk_idx / topk_logprob ([.][k], log-probabilities descending, e.g. from sage_expand_topk on the
 * draft model's logits of that node) holds node i's candidates; only frontier rows are read.
 * The call appends level l = depth(frontier) + 1: with alpha = alpha[alpha_row ? alpha_row[b] : b],
 * D = D(alpha), W = W(alpha) (Eq. 10, Eq. 11), W_1 = W and W_l = W / l * (0.5 + P_parent) beyond the
 * first level (P_parent = cumulative probability of the parent, 1 for the root), candidate rank r of
 * a frontier node joins iff r < W_l and its cumulative probability exceeds theta_l = 0.1 * l / D;
 * the scan of a row stops at the first rank that fails.  No level beyond D is opened.  Children are
 * appended in breadth-first order (parents by index, ranks ascending) until n_max nodes exist.
 * Afterwards frontier_begin[b] is the first new node and n_nodes[b] the new count; a call that finds
 * nothing to expand changes nothing.  The caller starts a tree with node 0 (parent -1, depth 0,
 * cum_logprob 0, its token), n_nodes = 1, frontier_begin = 0.  `policy` is a host pointer (its
 * thresholds are not used here).  d_max_seq, when not NULL, gives every sequence its own maximum
 * depth (e.g. from sage_update_history) in place of policy->d_max.  Decisions are taken in fp64 on
 * the fp32 inputs. */
int sage_grow_tree(const int32_t *topk_idx, const float *topk_logprob, int k,
                   const float *alpha, const int32_t *alpha_row, int batch,
                   const sage_tree_policy *policy, int n_max,
                   int32_t *parent, int32_t *rank, int32_t *depth, int32_t *token, float *cum_logprob,
                   int32_t *n_nodes, int32_t *frontier_begin,
                   const float *d_max_seq /* optional [batch]: replaces policy->d_max per sequence */,
                   int32_t *status, void *stream);

/* Adaptive history tracking (Section 3.3 "Adaptive History Tracking"; Section 5.1: window 10, lower
 * and upper thresholds 2 and 3).  Per sequence b: tau = path_len[b] - 1 (the acceptance length of the
 * round, from sage_accept) enters a sliding window of the last `window` values
 * (window_buf[b*window ..], count[b] = values pushed so far; the caller zeroes count once).  When at
 * least min_samples values are present and their mean is below `lower`, d_max[b] drops by `step`;
 * above `upper` it rises by `step`; in between it stays (hysteresis); always clamped to [d_lo, d_hi].
 * The paper fixes the window and the thresholds only; step, clamps and the warm-up rule are this
 * library's parameters.  d_max[b] can be fed to sage_grow_tree as the sequence's own maximum depth. */
typedef struct sage_history_policy {
    int   window;          /* paper: 10 */
    int   min_samples;     /* 1 .. window: no move before that many values */
    float lower, upper;    /* paper: 2, 3 */
    float step;            /* depth change per move */
    float d_lo, d_hi;      /* clamp range of d_max */
} sage_history_policy;
int sage_update_history(const int32_t *path_len, int batch, const sage_history_policy *policy /* host */,
                        int32_t *window_buf, int32_t *count, float *d_max,
                        int32_t *status, void *stream);

/* Tree attention mask as per-node ancestor bitsets (Section 2.2: each token attends
 * only to its ancestors; Algorithm 1 TreeAttnMask).  anc[i] has bit j set iff j == i or
 * j is an ancestor of i (local indices).  sage_tree_attention builds the same bitsets
 * internally; this entry point exposes them. */
int sage_build_ancestor_mask(const int32_t *parent, const int32_t *node_offsets, int batch,
                             uint64_t *anc, int32_t *status, void *stream);

/* Tree-masked verification attention (Section 2.2; Algorithm 1, the target model's
 * pass over all tree tokens with the mask; Section 3.3 "Phase 2").  For every layer,
 * sequence b, tree node i and query head h (KV head h / (n_q_heads/n_kv_heads)):
 *   out = softmax_t( sm_scale * q . K[t] ) V[t],  t over the prefix [0, L_b) and the tree
 *   slots L_b + j for j in anc(i).
 * q, out: bf16 [n_layers][sum_nodes][n_q_heads][head_dim]; `sum_nodes` is the node
 * capacity of those buffers (>= node_offsets[batch]).  Softmax and accumulation in
 * fp32.  Rows of the cache beyond L_b+N_b may hold anything (NaN included).
 * Rows of q and out beyond node_offsets[batch] are neither read nor written.  The work is scheduled from
 * the trees actually present, not from the capacity: where the host cannot tell which of the library's
 * kernels suits them (a long launch whose capacity allows trees of more than 128 query rows per KV
 * head), every candidate is started, each finds the largest tree of the batch in node_offsets on the
 * device, and all but the right one leave at once.
 * ws: sage_tree_attention_workspace_size(...) bytes: partial results of the sequences that a work
 * boundary or a context slice cuts (the larger of a fixed amount per streaming multiprocessor and an
 * amount per layer, context slice and query row). */
int sage_tree_attention(const void *q, const void *k_pool, const void *v_pool,
                        int64_t layer_stride_elems, int n_layers, int n_pages,
                        const int32_t *page_table, int max_pages_per_seq, const int32_t *seq_len,
                        const int32_t *parent, const int32_t *node_offsets, int batch, int sum_nodes,
                        int n_q_heads, int n_kv_heads, int head_dim, int page_size, float sm_scale,
                        void *out, void *ws, size_t ws_bytes, int32_t *status, void *stream);
size_t sage_tree_attention_workspace_size(int n_layers, int batch, int sum_nodes, int n_q_heads,
                                          int n_kv_heads, int head_dim, int max_pages_per_seq);

/* Greedy acceptance (Section 2.2: acceptance length = longest prefix matching the
 * target's predictions, Eq. 5; Section 3.3 "Phase 2").  Node c != root is accepted iff its
 * parent is accepted and draft_token[c] == target_argmax[parent[c]]; the root always is.
 * Among all root-to-leaf paths the one with the longest accepted prefix wins (cut at
 * max_path nodes); among equally long ones the lowest node index at the first point of
 * difference.  Writes path[b*max_path + j] (local node ids, -1 padded), path_len[b]
 * (= tau + 1) and bonus_token[b] = target_argmax at the last accepted node. */
int sage_accept(const int32_t *parent, const int32_t *draft_token, const int32_t *target_argmax,
                const int32_t *node_offsets, int batch, int max_path,
                int32_t *path, int32_t *path_len, int32_t *bonus_token,
                int32_t *status, void *stream);

/* KV-cache update with the accepted tokens (Algorithm 1; Section 3.3 "Phase 2").  In place,
 * for every layer, KV head and j < path_len[b]: the K and V rows at logical position
 * L_b + path[b][j] move to L_b + j (all rows are read before any is written), then
 * seq_len[b] += path_len[b].  No other byte of the pools changes.  A sequence whose path is not a
 * root path (entries not strictly increasing from 0, or path_len outside [0, max_path]) or whose
 * pages are out of range is reported in `status` and left untouched: no row moves and its
 * seq_len does not advance. */
int sage_compact_kv(void *k_pool, void *v_pool, int64_t layer_stride_elems, int n_layers, int n_pages,
                    const int32_t *page_table, int max_pages_per_seq, int32_t *seq_len,
                    const int32_t *path, const int32_t *path_len, int batch, int max_path,
                    int n_kv_heads, int head_dim, int page_size, int32_t *status, void *stream);

const char *sage_status_string(int code);

/* Diagnostics for the failure path of sage_tree_attention (no counterpart in the paper).  Every
 * on-device wait of that kernel has a cycle budget; when one runs out the thread block records
 * SAGE_STATUS_TIMEOUT, waits (again bounded) for its own copies and tensor-core work in flight,
 * releases its tensor memory and returns, so the context stays usable.  This call sets, for all
 * later sage_tree_attention calls of the process, the budget in clock cycles (<= 0 restores the
 * default of about two seconds) and, when producer_off != 0, keeps the copy warp from issuing
 * anything, so that the first consumer wait is one that nothing will ever satisfy.  Tests use it
 * to run the time-out path without faulting or hanging the device; leave it alone otherwise. */
void sage_debug_attention_waits(long long wait_cycles, int producer_off);

/* sage_tree_attention picks a schedule per launch: a streaming one (one resident thread block per
 * multiprocessor walks an equal share of all the work in steps of 128 keys; trees of up to 128 query
 * rows per KV head alternate their steps between two accumulator slots, trees of up to 256 keep two row
 * tiles per block) for long, HBM-bound launches, and a split one (a grid over context slices, row pairs
 * and KV heads, plus a merge) for tensor-bound trees and short launches.  schedule = 1 forces the
 * streaming one, 2 the split one, 3 the streaming one on two-block clusters that share every K/V tile
 * (one tensor-core instruction stream per cluster; measured slower, kept for comparison), anything
 * else restores the automatic choice.  For tests and measurements (no counterpart in the paper). */
void sage_debug_attention_schedule(int schedule);

#ifdef __cplusplus
}
#endif
#endif /* SAGE_H_ */
