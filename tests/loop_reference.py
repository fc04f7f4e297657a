"""CPU reference of the multi-round decode loop (Algorithm 1 with synthetic model stand-ins), built
from the oracle's functions only.  Test infrastructure: the device loop
(paper_2602_00523_b200.decode_loop) is compared with it round by round.

The stand-ins are the same data on both sides: the draft logits of every round, and the table of
pre-drawn agreement ranks (workloads.acceptance_picks) from which the target's greedy token per
node follows by a look-up.
"""
import numpy as np

import oracle
from workloads import NO_CANDIDATE

CAP = 64
MISS_TOKEN = 0


def target_tokens(picks_r, parent, rank, depth, n, draft_token, k):
    """The synthetic target's greedy token at every node of one tree (array of length n)."""
    child_of = {}
    for i in range(1, n):
        child_of[(int(parent[i]), int(rank[i]))] = i
    levels = picks_r.shape[1] - 1
    out = np.full(n, MISS_TOKEN, np.int32)
    for u in range(n):
        pick = int(picks_r[u, min(int(depth[u]) + 1, levels)])
        if pick != NO_CANDIDATE and pick < k and (u, pick) in child_of:
            out[u] = draft_token[child_of[(u, pick)]]
    return out


def reference_loop(policy, rounds, draft_logits, picks, k, k_entropy, max_path, trees=None, thresholds=(),
                   n_budget=CAP, levels=8, tree_policy_kw=None, history_kw=None, root_token=1, kv=None):
    """Returns per-round records (lists) and, when `kv` (dict with k_pool, v_pool, page_table, seq_len) is
    given, the final pools and sequence length.  `margin` is the smallest distance of any growth
    decision from its threshold (dynamic policy), so that a caller can insist on robust inputs."""
    tp = dict(d_min=3.0, d_max=8.0, w_min=2.0, w_max=10.0)
    tp.update(tree_policy_kw or {})
    hk = dict(window=10, lower=2.0, upper=3.0, step=1.0, d_lo=3.0, d_hi=8.0, min_samples=None)
    hk.update(history_kw or {})
    if hk["min_samples"] is None:
        hk["min_samples"] = hk["window"]
    window_buf = np.zeros(hk["window"], np.int32)
    count, d_max = 0, np.float32(tp["d_max"])
    alpha_prev = np.float32(0.5)
    root = np.int32(root_token)
    tid = 0
    rec = {n: [] for n in ("path_len", "n_nodes", "bonus", "d_max", "alpha", "template", "seq_len", "path",
                           "tree_parent", "draft_token")}
    if kv is not None:
        k_pool, v_pool, seq_len = kv["k_pool"].copy(), kv["v_pool"].copy(), kv["seq_len"].copy()
    for r in range(rounds):
        lg = draft_logits[r % len(draft_logits)]
        idx = oracle.topk(lg, k)
        _, lse = oracle.softmax_entropy(lg)
        lp = oracle.topk_logprob(lg, idx, lse).astype(np.float32)
        _, alpha = oracle.confidence(lg, k_entropy)
        if policy == "dynamic":
            parent = np.full(CAP, -1, np.int32); rank = np.zeros(CAP, np.int32); depth = np.zeros(CAP, np.int32)
            token = np.zeros(CAP, np.int32); cum = np.zeros(CAP, np.float32)
            token[0] = root
            n, fb = 1, 0
            for _ in range(levels):
                n, fb = oracle.grow_tree_level(parent, rank, depth, token, cum, n, fb, idx, lp, alpha_prev, n_max=n_budget,
                                               d_min=tp["d_min"], d_max=float(d_max), w_min=tp["w_min"], w_max=tp["w_max"])
            draft = token.copy()
        else:
            t = trees[tid]
            n = len(t["parent"])
            parent = np.full(CAP, -1, np.int32); rank = np.zeros(CAP, np.int32); depth = np.zeros(CAP, np.int32)
            parent[:n], rank[:n], depth[:n] = t["parent"], t["rank"], t["depth"]
            draft = np.zeros(CAP, np.int32)
            draft[:n] = oracle.expand_gather(idx, parent[:n], rank[:n], np.array([0, n]), np.array([root]))
        offs = np.array([0, n], np.int32)
        tgt = target_tokens(picks[r % len(picks)], parent, rank, depth, n, draft, k)
        path, plen, bonus = oracle.accept(parent[:n], draft[:n], tgt, offs, max_path)
        if kv is not None:
            k_pool, v_pool, seq_len = oracle.compact_kv(k_pool, v_pool, kv["page_table"], seq_len, path, plen, 64)
        count, d_max = oracle.update_history(window_buf, count, d_max, int(plen[0]) - 1, **hk)
        if policy == "templates":
            tid = int(oracle.select_tree(alpha[:1].astype(np.float32), list(thresholds))[0][0])
        rec["path_len"].append(int(plen[0])); rec["n_nodes"].append(n); rec["bonus"].append(int(bonus[0]))
        rec["d_max"].append(float(d_max)); rec["alpha"].append(float(alpha[0])); rec["template"].append(tid)
        rec["seq_len"].append(int(seq_len[0]) if kv is not None else 0); rec["path"].append(path[0].copy())
        rec["tree_parent"].append(parent.copy()); rec["draft_token"].append(draft.copy())
        alpha_prev = np.float32(alpha[0])
        root = np.int32(bonus[0])
    out = {"rec": rec}
    if kv is not None:
        out.update(k_pool=k_pool, v_pool=v_pool, seq_len=seq_len)
    return out
