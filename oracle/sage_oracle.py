"""fp64 NumPy oracle of the SAGE decode-round hot path.  TEST INFRASTRUCTURE ONLY.

Every function states the passage of the paper it follows.  Equation numbers
count the paper's displayed equations in order of appearance:
  Eq. 4  Top_k of the draft distribution at each depth      (Section 2.2)
  Eq. 5  best path p*                                        (Section 2.2)
  Eq. 7  top-k renormalisation                               (Section 3.1)
  Eq. 8  Shannon entropy of the renormalised distribution    (Section 3.1)
  Eq. 9  confidence alpha = 1 - H / log k                    (Section 3.1)
  Eq. 10 adaptive depth D(alpha)                             (Section 3.2)
  Eq. 11 adaptive width W(alpha)                             (Section 3.2)
Algorithm 1 is the overall inference pipeline (Section 3.3).

No blocking, fusion or reordering: each function is the definition written
out, with NumPy's matmul / sort as library steps.  Inputs are the same bytes
the CUDA library gets (bf16 bit patterns as uint16, fp32 logits), widened
exactly to fp64.
"""
from __future__ import annotations

import numpy as np


def widen_bf16(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp64, exactly."""
    return (np.asarray(bits).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------
# Tree attention mask  (Section 2.2: the mask lets a tree token see its
# ancestors only; Algorithm 1, TreeAttnMask).  A node also sees itself: the
# chain tree must reduce to ordinary causal attention, where a position sees
# itself.
# --------------------------------------------------------------------------
def ancestor_mask(parent: np.ndarray) -> np.ndarray:
    """anc[i] has bit j set iff j == i or j is an ancestor of i.  N <= 64."""
    parent = np.asarray(parent)
    n = len(parent)
    if n > 64:
        raise ValueError("at most 64 nodes (N_max of Section 5.1)")
    anc = np.zeros(n, dtype=np.uint64)
    for i in range(n):
        p = int(parent[i])
        if p < 0:
            anc[i] = np.uint64(1) << np.uint64(i)
        else:
            if not 0 <= p < i:
                raise ValueError("parent[i] must satisfy 0 <= parent[i] < i")
            anc[i] = anc[p] | (np.uint64(1) << np.uint64(i))
    return anc


# --------------------------------------------------------------------------
# Tree-masked verification attention  (Section 2.2; Algorithm 1, the target
# forward over all tree tokens with the mask M; Section 3.3 "Phase 2").
# --------------------------------------------------------------------------
def tree_attention(q_bits, k_pool_bits, v_pool_bits, page_table, seq_len, parent,
                   node_offsets, n_q_heads, n_kv_heads, head_dim, page_size, sm_scale):
    """Attention of every tree node against prefix + its ancestors, one layer.

    q_bits       uint16 [sumN, Hq, d]            bf16 queries of all tree nodes
    k/v_pool     uint16 [pages, Hkv, P, d]       paged bf16 cache of this layer
    page_table   int32  [B, max_pages]           logical page -> pool page
    seq_len      int32  [B]                      prefix length L_b; the tree's own
                                                 K/V sit at positions L_b .. L_b+N_b-1
    parent       int32  [sumN]                   local parent index per tree (-1 root)
    node_offsets int32  [B+1]
    Query head h uses KV head h // (Hq // Hkv).  Returns fp64 [sumN, Hq, d].
    """
    q = widen_bf16(q_bits)
    G = n_q_heads // n_kv_heads
    out = np.zeros((q.shape[0], n_q_heads, head_dim), dtype=np.float64)
    B = len(seq_len)
    for b in range(B):
        n0, n1 = int(node_offsets[b]), int(node_offsets[b + 1])
        N = n1 - n0
        L = int(seq_len[b])
        T = L + N
        anc = ancestor_mask(parent[n0:n1])
        # visible[i, t]: every prefix position; tree slot j iff j in anc(i)
        visible = np.zeros((N, T), dtype=bool)
        visible[:, :L] = True
        for i in range(N):
            for j in range(N):
                if (int(anc[i]) >> j) & 1:
                    visible[i, L + j] = True
        pos = np.arange(T)
        pages = np.asarray(page_table[b])[pos // page_size]
        slots = pos % page_size
        for g in range(n_kv_heads):
            K = widen_bf16(k_pool_bits[pages, g, slots, :])      # [T, d]
            Vv = widen_bf16(v_pool_bits[pages, g, slots, :])     # [T, d]
            for hg in range(G):
                h = g * G + hg
                s = sm_scale * (q[n0:n1, h, :] @ K.T)            # [N, T]
                s = np.where(visible, s, -np.inf)
                s = s - s.max(axis=1, keepdims=True)
                p = np.exp(s)
                p = p / p.sum(axis=1, keepdims=True)
                out[n0:n1, h, :] = p @ Vv
    return out


# --------------------------------------------------------------------------
# Row-wise softmax entropy over the whole vocabulary (Eq. 8 applied to the
# full distribution P = softmax(logits), Eq. 1), natural log.
# --------------------------------------------------------------------------
def softmax_entropy(logits: np.ndarray):
    """Returns (H_full [rows], lse [rows]) in fp64.  H = lse - sum p*x."""
    x = np.asarray(logits).astype(np.float64)
    m = x.max(axis=1, keepdims=True)
    e = np.exp(x - m)
    s = e.sum(axis=1, keepdims=True)
    p = e / s
    lse = (m + np.log(s))[:, 0]
    with np.errstate(divide="ignore", invalid="ignore"):
        plogp = np.where(p > 0, p * np.log(p), 0.0)
    return -plogp.sum(axis=1), lse


# --------------------------------------------------------------------------
# Top-k  (Eq. 4).  Order: value descending, ties to the lowest index.
# --------------------------------------------------------------------------
def topk(logits: np.ndarray, k: int) -> np.ndarray:
    """Indices [rows, k] of the k largest entries, sorted (value desc, index asc)."""
    x = np.asarray(logits).astype(np.float64) + 0.0   # -0.0 + 0.0 = +0.0
    order = np.argsort(-x, axis=1, kind="stable")      # stable: equal values keep index order
    return order[:, :k].astype(np.int32)


def topk_logprob(logits: np.ndarray, idx: np.ndarray, lse: np.ndarray) -> np.ndarray:
    """log P of the selected entries: x - logsumexp(x)."""
    x = np.asarray(logits).astype(np.float64)
    return np.take_along_axis(x, idx.astype(np.int64), axis=1) - lse[:, None]


# --------------------------------------------------------------------------
# Confidence  (Eq. 7, Eq. 8, Eq. 9)
# --------------------------------------------------------------------------
def confidence(logits: np.ndarray, k_entropy: int):
    """(H_topk [rows], alpha [rows]): entropy of the renormalised top-k, and
    alpha = 1 - H / ln k clamped to [0, 1] (alpha = 1 when k = 1)."""
    x = np.asarray(logits).astype(np.float64)
    idx = topk(logits, k_entropy).astype(np.int64)
    top = np.take_along_axis(x, idx, axis=1)
    # P_i / sum_{j in top-k} P_j: the softmax normaliser cancels
    w = np.exp(top - top[:, :1])
    pt = w / w.sum(axis=1, keepdims=True)
    with np.errstate(divide="ignore", invalid="ignore"):
        H = -np.where(pt > 0, pt * np.log(pt), 0.0).sum(axis=1)
    if k_entropy == 1:
        alpha = np.ones_like(H)
    else:
        alpha = np.clip(1.0 - H / np.log(float(k_entropy)), 0.0, 1.0)
    return H, alpha


# --------------------------------------------------------------------------
# Depth / width from alpha  (Eq. 10, Eq. 11; Algorithm 1 "Phase 3").  The
# paper leaves the mapping from the real-valued (D, W) to a concrete tree
# open; here a tree template is picked by comparing alpha with descending
# thresholds.  The comparison is done on the fp32 alpha it is handed, in
# fp32: alpha arrives as an fp32 array (the storage type of the confidence
# outputs), and comparing it in any wider type against thresholds that are
# themselves fp32 policy constants would decide a different question.
# --------------------------------------------------------------------------
def select_tree(alpha, thresholds, d_min=3.0, d_max=8.0, w_min=2.0, w_max=10.0):
    """Returns (template_id int32 [B], D_cont fp64 [B], W_cont fp64 [B]).
    template_id = number of thresholds strictly above alpha."""
    a32 = np.asarray(alpha, dtype=np.float32)
    thr = np.asarray(thresholds, dtype=np.float32)
    tid = np.zeros(a32.shape, dtype=np.int32)
    for t in thr:
        tid += (a32 < t).astype(np.int32)
    a = a32.astype(np.float64)
    D = d_min + a * (d_max - d_min)
    W = w_min + (1.0 - a) * (w_max - w_min)
    return tid, D, W


# --------------------------------------------------------------------------
# Draft-node expansion  (Section 2.2 "Tree-based Drafting"; Section 3.2
# "Dynamic Tree Construction": a node's children carry the top candidates of
# its output distribution)
# --------------------------------------------------------------------------
def expand_gather(topk_idx, parent, rank, node_offsets, root_token):
    """draft_token[i] = topk_idx[row of parent(i)][rank[i]]; roots get root_token[b].
    Logits row r belongs to global node r."""
    topk_idx = np.asarray(topk_idx)
    out = np.zeros(len(parent), dtype=np.int32)
    for b in range(len(node_offsets) - 1):
        n0, n1 = int(node_offsets[b]), int(node_offsets[b + 1])
        for i in range(n0, n1):
            p = int(parent[i])
            out[i] = root_token[b] if p < 0 else topk_idx[n0 + p, int(rank[i])]
    return out


# --------------------------------------------------------------------------
# Greedy acceptance  (Section 2.2: the acceptance length tau is that of the
# longest prefix agreeing with the target's own predictions, and tau + 1 tokens
# are committed; Eq. 5; Section 3.3 "Phase 2": every draft token on the chosen
# path equals the target's greedy output at its parent).
# --------------------------------------------------------------------------
def accept(parent, draft_token, target_argmax, node_offsets, max_path):
    """Best path by enumeration of every root-to-leaf path.

    A path root = v_0, v_1, ..., v_m is accepted up to the first l with
    draft_token[v_l] != target_argmax[v_{l-1}] (the root, the last committed
    token, is always accepted); its accepted prefix is cut at max_path nodes.
    The path with the longest accepted prefix wins; among equally long ones the
    prefix that is lexicographically smallest as a list of node indices.
    Returns (path [B, max_path] local node ids, -1 padded; path_len [B] =
    tau + 1; bonus [B] = target_argmax at the last accepted node)."""
    B = len(node_offsets) - 1
    path = np.full((B, max_path), -1, dtype=np.int32)
    path_len = np.zeros(B, dtype=np.int32)
    bonus = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n0, n1 = int(node_offsets[b]), int(node_offsets[b + 1])
        par = [int(v) for v in parent[n0:n1]]
        tok = [int(v) for v in draft_token[n0:n1]]
        tgt = [int(v) for v in target_argmax[n0:n1]]
        n = n1 - n0
        has_child = [False] * n
        for i in range(1, n):
            has_child[par[i]] = True
        best = None
        for leaf in range(n):
            if has_child[leaf]:
                continue
            nodes = []
            c = leaf
            while c >= 0:
                nodes.append(c)
                c = par[c]
            nodes.reverse()
            m = 1
            while m < len(nodes) and m < max_path and tok[nodes[m]] == tgt[nodes[m - 1]]:
                m += 1
            prefix = nodes[:m]
            if best is None or len(prefix) > len(best) or (len(prefix) == len(best) and prefix < best):
                best = prefix
        path[b, :len(best)] = best
        path_len[b] = len(best)
        bonus[b] = tgt[best[-1]]
    return path, path_len, bonus


# --------------------------------------------------------------------------
# KV-cache update with the accepted tokens  (Algorithm 1, the cache-update
# step that follows the acceptance step; Section 3.3 "Phase 2")
# --------------------------------------------------------------------------
def compact_kv(k_pool, v_pool, page_table, seq_len, path, path_len, page_size):
    """For every layer and KV head move the row at logical position
    L_b + path[b][j] to L_b + j (j < path_len[b]); seq_len += path_len.
    Pools are uint16 [layers, pages, Hkv, P, d]; returns new (k, v, seq_len)."""
    k_new, v_new = k_pool.copy(), v_pool.copy()
    new_len = np.asarray(seq_len).copy()
    for b in range(len(seq_len)):
        L = int(seq_len[b])
        for j in range(int(path_len[b])):
            src = L + int(path[b][j])
            dst = L + j
            sp, ss = int(page_table[b][src // page_size]), src % page_size
            dp, ds = int(page_table[b][dst // page_size]), dst % page_size
            # read from the untouched input pools: all sources are gathered before any write
            k_new[:, dp, :, ds, :] = k_pool[:, sp, :, ss, :]
            v_new[:, dp, :, ds, :] = v_pool[:, sp, :, ss, :]
        new_len[b] = L + int(path_len[b])
    return k_new, v_new, new_len


# --------------------------------------------------------------------------
# Dynamic tree construction, one level at a time  (Section 3.2: "Hierarchical
# Width Decay", Eq. 12, and "Dynamic Tree Construction").  A path is in the tree
# iff at every level l its rank p_l < W_l and its cumulative probability exceeds
# theta_l = 0.1 * l / D(alpha); W_1 = W(alpha), and beyond the first level
# W_l = W(alpha) / l * (0.5 + P_parent).  Readings taken where the paper is
# silent: P_parent is the cumulative path probability of the parent (1 for the
# root); "p_l < W_l" is used as it stands with the real-valued W_l (no rounding
# rule is invented); a level l exists iff l <= D(alpha); nodes are added in
# breadth-first order (parents by index, ranks ascending) until N_max nodes.
# Decisions are taken in fp64 on the fp32 inputs; cumulative log-probabilities
# are fp32 sums, because fp32 is the storage type of the log-probabilities the
# caller hands over and of the per-node array the sums are kept in from one
# level to the next.  "parity unpinned" for these
# readings; the level-wise construction itself is pinned against the path rule
# evaluated directly on every path of a full k-ary tree.
# --------------------------------------------------------------------------
def grow_tree_level(parent, rank, depth, token, cum_logprob, n_nodes, frontier_begin,
                    topk_idx, topk_logprob, alpha, n_max=64,
                    d_min=3.0, d_max=8.0, w_min=2.0, w_max=10.0):
    """Adds the next level to one tree (arrays of capacity >= n_max, modified in place).

    Nodes frontier_begin .. n_nodes-1 are the deepest level so far; row i of topk_idx /
    topk_logprob holds node i's k best next tokens and their log-probabilities (descending).
    Returns (new n_nodes, new frontier_begin)."""
    a = float(np.float32(alpha))
    D = d_min + a * (d_max - d_min)
    W = w_min + (1.0 - a) * (w_max - w_min)
    k = topk_idx.shape[1]
    n = int(n_nodes)
    if n <= int(frontier_begin):
        return n, int(frontier_begin)
    level = int(depth[int(frontier_begin)]) + 1
    new_begin = n
    if float(level) > D:
        return n, new_begin
    theta = 0.1 * level / D
    for u in range(int(frontier_begin), int(n_nodes)):
        p_parent = float(np.exp(np.float64(cum_logprob[u])))
        w_l = W if level == 1 else W / level * (0.5 + p_parent)
        for r in range(k):
            if not (float(r) < w_l):
                break
            c = np.float32(np.float32(cum_logprob[u]) + np.float32(topk_logprob[u, r]))
            if not (float(np.exp(np.float64(c))) > theta):
                break
            if n >= n_max:
                return n, new_begin
            parent[n], rank[n], depth[n] = u, r, level
            token[n], cum_logprob[n] = topk_idx[u, r], c
            n += 1
    return n, new_begin


# --------------------------------------------------------------------------
# Adaptive history tracking  (Section 3.3 "Adaptive History Tracking"; window
# size 10 and thresholds 2 / 3 in Section 5.1 "Implementation details").  A
# sliding window of recent acceptance lengths tau; when their mean falls below
# the lower threshold the maximum depth goes down, above the upper threshold it
# goes up, in between it stays.  The paper gives neither the step nor the
# clamps nor what happens before the window is full: here the step and the
# clamp range are parameters, and nothing moves until `min_samples` values are
# in the window ("parity unpinned" for those readings).
# --------------------------------------------------------------------------
def update_history(window_buf, count, d_max, tau, window=10, lower=2.0, upper=3.0, step=1.0,
                   d_lo=3.0, d_hi=8.0, min_samples=10):
    """One sequence: pushes tau into the ring `window_buf` (int32 [window], in place) and returns
    (new count, new d_max)."""
    window_buf[int(count) % window] = int(tau)
    count = int(count) + 1
    n = min(count, window)
    d = float(np.float32(d_max))
    if n >= min_samples:
        mean = float(np.sum(window_buf[:n].astype(np.int64))) / n
        if mean < lower:
            d = max(float(d_lo), d - float(step))
        elif mean > upper:
            d = min(float(d_hi), d + float(step))
    return count, np.float32(d)


def expected_acceptance_length(p, gamma, depth):
    """Closed form of Theorem 2 (Section 4.2): E[tau] = sum_{l=1..D} p^l gamma^(l(l-1)/2) for greedy-path
    speculation whose level-l token is accepted with probability p gamma^(l-1)."""
    return float(sum(p ** l * gamma ** (l * (l - 1) / 2.0) for l in range(1, int(depth) + 1)))
