"""Pins for the oracle's dynamic tree construction (Section 3.2, Eq. 12 and "Dynamic Tree
Construction").  The level-by-level builder is checked against the paper's path rule evaluated
directly, path by path, on the full k-ary tree; closed-form cases cover the width decay, the
probability threshold, the depth limit and the node budget."""
import itertools

import numpy as np

import oracle


def node_rows(rng, k):
    """Top-k log-probabilities of one node: a descending row that sums to less than 1 in probability."""
    p = np.sort(rng.dirichlet(np.ones(k + 3) * 0.6))[::-1][:k]
    return np.log(p).astype(np.float32)


class LazyTree:
    """Per-path top-k rows, drawn on first use from a seed and the path."""
    def __init__(self, seed, k):
        self.seed, self.k, self.rows = seed, k, {}

    def row(self, path):
        if path not in self.rows:
            h = np.random.Generator(np.random.Philox([self.seed, hash(path) & 0xFFFFFFFF]))
            self.rows[path] = node_rows(h, self.k)
        return self.rows[path]


def build_levelwise(lazy, alpha, n_max, cap=4096, **policy):
    k = lazy.k
    parent = np.full(cap, -1, np.int32); rank = np.zeros(cap, np.int32); depth = np.zeros(cap, np.int32)
    token = np.zeros(cap, np.int32); cum = np.zeros(cap, np.float32)
    topk_idx = np.zeros((cap, k), np.int32); topk_lp = np.zeros((cap, k), np.float32)
    paths = {0: ()}
    n, fb = 1, 0
    while True:
        for u in range(fb, n):
            topk_lp[u] = lazy.row(paths[u])
            topk_idx[u] = np.arange(k) + 100 * u
        n2, fb2 = oracle.grow_tree_level(parent, rank, depth, token, cum, n, fb, topk_idx, topk_lp, alpha,
                                         n_max=n_max, **policy)
        for i in range(n, n2):
            paths[i] = paths[int(parent[i])] + (int(rank[i]),)
        if n2 == n:
            break
        n, fb = n2, fb2
    return n, parent[:n].copy(), rank[:n].copy(), depth[:n].copy(), cum[:n].copy(), [paths[i] for i in range(n)]


def paths_by_rule(lazy, alpha, d_min=3.0, d_max=8.0, w_min=2.0, w_max=10.0):
    """The paper's rule, path by path: included iff at every level l the rank p_l < W_l and the
    cumulative probability exceeds theta_l."""
    a = float(np.float32(alpha))
    D = d_min + a * (d_max - d_min)
    W = w_min + (1 - a) * (w_max - w_min)
    out = set()
    for d in range(1, int(np.floor(D)) + 1):
        for path in itertools.product(range(lazy.k), repeat=d):
            cum = np.float32(0.0)
            ok = True
            for l in range(1, d + 1):
                p_parent = float(np.exp(np.float64(cum)))
                w_l = W if l == 1 else W / l * (0.5 + p_parent)
                cum = np.float32(cum + lazy.row(path[:l - 1])[path[l - 1]])
                if not (path[l - 1] < w_l and float(np.exp(np.float64(cum))) > 0.1 * l / D):
                    ok = False
                    break
            if ok:
                out.add(path)
    return out


def test_levelwise_builder_equals_the_path_rule_on_full_trees():
    for seed, alpha, k in [(1, 0.0, 3), (2, 0.3, 3), (3, 0.6, 4), (4, 0.05, 4), (5, 0.9, 3)]:
        lazy = LazyTree(seed, k)
        policy = dict(d_min=2.0, d_max=4.0, w_min=1.5, w_max=4.0)
        n, parent, rank, depth, cum, paths = build_levelwise(lazy, alpha, n_max=4096, **policy)
        want = paths_by_rule(lazy, alpha, **policy)
        assert set(paths[1:]) == want, (seed, alpha)
        assert len(set(paths)) == n                       # no duplicates
        assert all(parent[i] < i for i in range(1, n)) and list(depth) == sorted(depth)


def test_first_level_width_and_decay_closed_forms():
    # alpha = 1: W = 2, D = 8.  Level 1 takes ranks 0 and 1; at level 2, W_2 = (0.5 + P_parent), so
    # rank 0 always passes the width test and rank 1 only if P_parent > 0.5.
    k = 4
    row_root = np.log(np.array([0.7, 0.25, 0.03, 0.02], np.float32))
    row_any = np.log(np.array([0.9, 0.05, 0.03, 0.02], np.float32))
    cap = 64
    parent = np.full(cap, -1, np.int32); rank = np.zeros(cap, np.int32); depth = np.zeros(cap, np.int32)
    token = np.zeros(cap, np.int32); cum = np.zeros(cap, np.float32)
    idx = np.tile(np.arange(k, dtype=np.int32), (cap, 1)); lp = np.tile(row_any, (cap, 1)); lp[0] = row_root
    n, fb = oracle.grow_tree_level(parent, rank, depth, token, cum, 1, 0, idx, lp, 1.0)
    assert (n, fb) == (3, 1) and list(rank[1:3]) == [0, 1]
    assert np.allclose(np.exp(cum[1:3]), [0.7, 0.25])
    n2, fb2 = oracle.grow_tree_level(parent, rank, depth, token, cum, n, fb, idx, lp, 1.0)
    # node 1 (P = 0.7 > 0.5): ranks 0 and 1 pass the width test; rank 1 has P = 0.035 > theta_2 = 0.025
    # node 2 (P = 0.25): W_2 = 0.75 -> rank 0 only
    assert fb2 == 3 and [(int(parent[i]), int(rank[i])) for i in range(3, n2)] == [(1, 0), (1, 1), (2, 0)]


def test_probability_threshold_depth_limit_and_node_budget():
    k = 3
    cap = 64
    idx = np.tile(np.arange(k, dtype=np.int32), (cap, 1))

    def fresh():
        return (np.full(cap, -1, np.int32), np.zeros(cap, np.int32), np.zeros(cap, np.int32),
                np.zeros(cap, np.int32), np.zeros(cap, np.float32))
    # alpha = 0: W = 10, D = 3, theta_1 = 0.1/3.  A candidate at exactly-below-threshold probability stops the row.
    lp = np.tile(np.log(np.array([0.5, 0.03, 0.4], np.float32)), (cap, 1))   # not sorted on purpose: rank 1 fails
    arrs = fresh()
    n, fb = oracle.grow_tree_level(*arrs, 1, 0, idx, lp, 0.0)
    assert n == 2                                      # rank 0 only: the scan stops at the first failing rank
    # depth limit: with D = 3 a fourth level never appears
    lp = np.tile(np.log(np.array([0.98, 0.01, 0.005], np.float32)), (cap, 1))
    arrs = fresh()
    n, fb = 1, 0
    for _ in range(6):
        n, fb = oracle.grow_tree_level(*arrs, n, fb, idx, lp, 0.0)
    assert int(arrs[2][:n].max()) == 3
    # node budget: the truncated tree is a breadth-first prefix of the untruncated one
    lp = np.tile(np.log(np.array([0.4, 0.35, 0.2], np.float32)), (cap, 1))
    full = fresh()
    n, fb = 1, 0
    for _ in range(4):
        n, fb = oracle.grow_tree_level(*full, n, fb, idx, lp, 0.0, n_max=64)
    cut = fresh()
    m, fb = 1, 0
    for _ in range(4):
        m, fb = oracle.grow_tree_level(*cut, m, fb, idx, lp, 0.0, n_max=7)
    assert m == 7 and n > 7
    assert np.array_equal(cut[0][:7], full[0][:7]) and np.array_equal(cut[1][:7], full[1][:7])
