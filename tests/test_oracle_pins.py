"""Pins for the CPU oracle: each oracle function is checked against something
other than itself -- brute force in pure Python, closed forms, invariants,
library routines, and the few values the paper fixes."""
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle
from workloads import (bf16_bits, bf16_to_f32, chain_tree, make_kv_cache, make_q, make_template,
                       random_tree, star_tree, TEMPLATES)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


# ---------------------------------------------------------------- ancestors
def brute_ancestors(parent, i):
    s = set()
    while i >= 0:
        s.add(i)
        i = int(parent[i])
    return s


@pytest.mark.parametrize("seed", range(5))
def test_ancestor_mask_brute_force(seed):
    t = random_tree(rng(seed), 2 + 7 * seed if seed else 1)
    anc = oracle.ancestor_mask(t["parent"])
    for i in range(len(anc)):
        bits = {j for j in range(64) if (int(anc[i]) >> j) & 1}
        assert bits == brute_ancestors(t["parent"], i)


def test_ancestor_mask_chain_star_and_limits():
    anc = oracle.ancestor_mask(chain_tree(64)["parent"])
    for i in range(64):
        assert int(anc[i]) == (1 << (i + 1)) - 1          # lower-triangular (causal) mask
    anc = oracle.ancestor_mask(star_tree(10)["parent"])
    assert int(anc[0]) == 1
    for i in range(1, 10):
        assert int(anc[i]) == (1 | (1 << i))
    with pytest.raises(ValueError):
        oracle.ancestor_mask(np.array([-1] + [0] * 64))
    with pytest.raises(ValueError):
        oracle.ancestor_mask(np.array([-1, 2, 0]))


# ---------------------------------------------------------------- attention
def tiny_attention_case(seed, tree, L=5, Hq=4, Hkv=2, d=8, P=4, shuffle=True):
    r = rng(100 + seed)
    N = len(tree["parent"])
    kv = make_kv_cache(r, [L], [N], [L // 2], Hkv, head_dim=d, page_size=P, shuffle=shuffle,
                       spare_frac=0.5 if shuffle else 0.0)
    q = make_q(r, N, Hq, d)[0]
    return q, kv


def brute_dense_attention(q, kv, tree, L, Hq, Hkv, d, P, scale):
    """Pure-Python loops: explicit additive mask over L+N keys, softmax, weighted sum."""
    parent = tree["parent"]
    N = len(parent)
    T = L + N
    G = Hq // Hkv
    qf = bf16_to_f32(q).astype(np.float64)
    kf = bf16_to_f32(kv["k_pool"][0]).astype(np.float64)
    vf = bf16_to_f32(kv["v_pool"][0]).astype(np.float64)
    pt = kv["page_table"][0]
    out = np.zeros((N, Hq, d))
    for i in range(N):
        allowed = brute_ancestors(parent, i)
        add_mask = [0.0 if (t < L or (t - L) in allowed) else -math.inf for t in range(T)]
        for h in range(Hq):
            g = h // G
            scores = []
            for t in range(T):
                kr = kf[pt[t // P], g, t % P]
                dot = 0.0
                for c in range(d):
                    dot += qf[i, h, c] * kr[c]
                scores.append(dot * scale + add_mask[t])
            mx = max(scores)
            w = [math.exp(s - mx) for s in scores]
            z = sum(w)
            for t in range(T):
                vr = vf[pt[t // P], g, t % P]
                for c in range(d):
                    out[i, h, c] += w[t] / z * vr[c]
    return out


def run_oracle_attention(q, kv, tree, Hq, Hkv, d, P, scale):
    N = len(tree["parent"])
    return oracle.tree_attention(q, kv["k_pool"][0], kv["v_pool"][0], kv["page_table"], kv["seq_len"],
                                 tree["parent"], np.array([0, N], dtype=np.int32), Hq, Hkv, d, P, scale)


@pytest.mark.parametrize("seed", range(3))
def test_attention_vs_brute_force_dense_mask(seed):
    tree = random_tree(rng(seed), 6)
    q, kv = tiny_attention_case(seed, tree)
    got = run_oracle_attention(q, kv, tree, 4, 2, 8, 4, 0.37)
    want = brute_dense_attention(q, kv, tree, 5, 4, 2, 8, 4, 0.37)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_attention_chain_tree_is_causal_attention():
    N, L, Hq, Hkv, d, P = 7, 9, 4, 2, 8, 4
    tree = chain_tree(N)
    q, kv = tiny_attention_case(7, tree, L=L)
    got = run_oracle_attention(q, kv, tree, Hq, Hkv, d, P, 0.5)
    # independent statement: node i is position L+i of a causal sequence
    pt = kv["page_table"][0]
    pos = np.arange(L + N)
    qf = bf16_to_f32(q).astype(np.float64)
    for h in range(Hq):
        g = h // (Hq // Hkv)
        K = bf16_to_f32(kv["k_pool"][0][pt[pos // P], g, pos % P]).astype(np.float64)
        V = bf16_to_f32(kv["v_pool"][0][pt[pos // P], g, pos % P]).astype(np.float64)
        for i in range(N):
            w = scipy.special.softmax(0.5 * (K[:L + i + 1] @ qf[i, h]))
            np.testing.assert_allclose(got[i, h], w @ V[:L + i + 1], rtol=1e-12, atol=1e-13)


def test_attention_single_node_is_plain_decode():
    tree = chain_tree(1)
    q, kv = tiny_attention_case(3, tree, L=11)
    got = run_oracle_attention(q, kv, tree, 4, 2, 8, 4, 0.25)
    pt = kv["page_table"][0]
    pos = np.arange(12)
    qf = bf16_to_f32(q).astype(np.float64)
    for h in range(4):
        K = bf16_to_f32(kv["k_pool"][0][pt[pos // 4], h // 2, pos % 4]).astype(np.float64)
        V = bf16_to_f32(kv["v_pool"][0][pt[pos // 4], h // 2, pos % 4]).astype(np.float64)
        np.testing.assert_allclose(got[0, h], scipy.special.softmax(0.25 * K @ qf[0, h]) @ V, rtol=1e-12)


def test_attention_non_ancestor_perturbation_and_page_permutation():
    tree = random_tree(rng(11), 8)
    L, P = 6, 4
    q, kv = tiny_attention_case(11, tree, L=L, shuffle=False)
    base = run_oracle_attention(q, kv, tree, 4, 2, 8, P, 0.3)
    # change K/V of tree slot j: only nodes having j as ancestor-or-self may move
    j = 3
    kv2 = {k: v.copy() for k, v in kv.items()}
    t = L + j
    kv2["k_pool"][0, kv["page_table"][0][t // P], :, t % P, :] = bf16_bits(np.full((2, 8), 3.0, np.float32))
    kv2["v_pool"][0, kv["page_table"][0][t // P], :, t % P, :] = bf16_bits(np.full((2, 8), -2.0, np.float32))
    pert = run_oracle_attention(q, kv2, tree, 4, 2, 8, P, 0.3)
    for i in range(8):
        if j in brute_ancestors(tree["parent"], i):
            assert np.abs(pert[i] - base[i]).max() > 1e-6
        else:
            np.testing.assert_array_equal(pert[i], base[i])
    # permute the physical pages: same logical cache, same answer
    n_pages = kv["k_pool"].shape[1]
    perm = rng(5).permutation(n_pages)
    kv3 = {k: v.copy() for k, v in kv.items()}
    kv3["k_pool"][0, perm] = kv["k_pool"][0]
    kv3["v_pool"][0, perm] = kv["v_pool"][0]
    kv3["page_table"] = perm[kv["page_table"]].astype(np.int32)
    np.testing.assert_array_equal(run_oracle_attention(q, kv3, tree, 4, 2, 8, P, 0.3), base)


def test_attention_equal_keys_gives_mean_of_visible_values():
    tree = random_tree(rng(2), 5)
    L, P = 4, 4
    q, kv = tiny_attention_case(2, tree, L=L, shuffle=False)
    kv["k_pool"][:] = bf16_bits(np.float32([0.5]))[0]
    got = run_oracle_attention(q, kv, tree, 4, 2, 8, P, 0.3)
    vf = bf16_to_f32(kv["v_pool"][0]).astype(np.float64)
    pt = kv["page_table"][0]
    for i in range(5):
        vis = list(range(L)) + [L + j for j in sorted(brute_ancestors(tree["parent"], i))]
        for h in range(4):
            rows = np.stack([vf[pt[t // P], h // 2, t % P] for t in vis])
            np.testing.assert_allclose(got[i, h], rows.mean(axis=0), rtol=1e-12, atol=1e-14)


def test_attention_batch_is_per_sequence():
    r = rng(77)
    trees = [random_tree(r, 4), random_tree(r, 6)]
    kv = make_kv_cache(r, [5, 9], [4, 6], [2, 3], 2, head_dim=8, page_size=4, shuffle=True, spare_frac=0.3)
    q = make_q(r, 10, 4, 8)[0]
    parent = np.concatenate([t["parent"] for t in trees])
    offs = np.array([0, 4, 10], dtype=np.int32)
    both = oracle.tree_attention(q, kv["k_pool"][0], kv["v_pool"][0], kv["page_table"], kv["seq_len"],
                                 parent, offs, 4, 2, 8, 4, 0.4)
    for b, (n0, n1) in enumerate([(0, 4), (4, 10)]):
        one = oracle.tree_attention(q[n0:n1], kv["k_pool"][0], kv["v_pool"][0], kv["page_table"][b:b + 1],
                                    kv["seq_len"][b:b + 1], trees[b]["parent"],
                                    np.array([0, n1 - n0], dtype=np.int32), 4, 2, 8, 4, 0.4)
        want = brute_dense_attention(q[n0:n1], {"k_pool": kv["k_pool"], "v_pool": kv["v_pool"],
                                                "page_table": kv["page_table"][b:b + 1]},
                                     trees[b], int(kv["seq_len"][b]), 4, 2, 8, 4, 0.4)
        np.testing.assert_array_equal(both[n0:n1], one)
        np.testing.assert_allclose(one, want, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- entropy
def test_entropy_closed_forms():
    V = 152064
    H, lse = oracle.softmax_entropy(np.full((2, V), 3.25, np.float32))
    np.testing.assert_allclose(H, math.log(V), atol=1e-10)
    np.testing.assert_allclose(lse, 3.25 + math.log(V), atol=1e-10)
    x = np.zeros((1, V), np.float32)
    x[0, 777] = 1e4
    H, lse = oracle.softmax_entropy(x)
    assert abs(H[0]) < 1e-12 and abs(lse[0] - 1e4) < 1e-9
    # a entries at c, the rest at 0:  Z = a e^c + V - a,  H = ln Z - a c e^c / Z
    for a, c in [(1, 5.0), (10, 9.5), (1000, -2.0)]:
        x = np.zeros((1, V), np.float32)
        x[0, 5:5 + a] = c
        Z = a * math.exp(c) + V - a
        H, lse = oracle.softmax_entropy(x)
        np.testing.assert_allclose(H[0], math.log(Z) - a * c * math.exp(c) / Z, rtol=1e-12)
        np.testing.assert_allclose(lse[0], math.log(Z), rtol=1e-12)


def test_entropy_vs_library_routine():
    x = rng(1).standard_normal((4, 5000)).astype(np.float32) * np.float32([[0.5], [1], [4], [12]])
    H, lse = oracle.softmax_entropy(x)
    p = scipy.special.softmax(x.astype(np.float64), axis=1)
    np.testing.assert_allclose(H, scipy.stats.entropy(p, axis=1), rtol=1e-11)
    np.testing.assert_allclose(lse, scipy.special.logsumexp(x.astype(np.float64), axis=1), rtol=1e-13)


# ---------------------------------------------------------------- top-k
def brute_topk(row, k):
    return [i for i, _ in sorted(enumerate(row), key=lambda t: (-float(t[1]), t[0]))][:k]


def test_topk_brute_force_and_ties():
    r = rng(3)
    x = r.integers(-3, 4, size=(6, 40)).astype(np.float32)       # many exact ties
    x[2, 7] = -0.0
    x[2, 3] = 0.0
    for k in (1, 4, 16, 40):
        got = oracle.topk(x, k)
        for i in range(6):
            assert list(got[i]) == brute_topk(x[i], k)
    np.testing.assert_array_equal(oracle.topk(np.full((2, 100), 1.5, np.float32), 10),
                                  np.tile(np.arange(10), (2, 1)))
    # -0.0 and +0.0 compare equal: the lower index wins whatever the sign
    z = np.full((1, 8), -1.0, np.float32)
    z[0, 2], z[0, 5] = 0.0, -0.0
    assert list(oracle.topk(z, 2)[0]) == [2, 5]
    z[0, 2], z[0, 5] = -0.0, 0.0
    assert list(oracle.topk(z, 2)[0]) == [2, 5]


def test_topk_logprob_sums_to_one_over_full_row():
    x = rng(4).standard_normal((3, 64)).astype(np.float32)
    _, lse = oracle.softmax_entropy(x)
    lp = oracle.topk_logprob(x, oracle.topk(x, 64), lse)
    np.testing.assert_allclose(np.exp(lp).sum(axis=1), 1.0, rtol=1e-12)
    assert (np.diff(lp, axis=1) <= 0).all()


# ---------------------------------------------------------------- confidence
def max_entropy_given_p1(p1, k):
    """Largest entropy of a k-point distribution whose top probability is p1 (first
    step of the proof of Lemma 1): the other k-1 entries share 1-p1 evenly."""
    if p1 >= 1.0:
        return 0.0
    return -p1 * math.log(p1) - (1 - p1) * math.log((1 - p1) / (k - 1))


def test_confidence_endpoints_and_base_independence():
    V, k = 1000, 10
    x = np.full((1, V), -50.0, np.float32)
    x[0, 100:110] = 2.0                                    # uniform over the top-k
    H, a = oracle.confidence(x, k)
    np.testing.assert_allclose(H[0], math.log(k), rtol=1e-13)
    assert abs(a[0]) < 1e-13
    x = rng(5).standard_normal((1, V)).astype(np.float32)
    x[0, 3] = 1e3                                          # one dominant entry
    H, a = oracle.confidence(x, k)
    assert abs(H[0]) < 1e-12 and a[0] == 1.0
    _, a1 = oracle.confidence(x, 1)
    assert a1[0] == 1.0
    # log base does not matter: alpha = 1 - H_base_k
    x = rng(6).standard_normal((5, V)).astype(np.float32) * 2
    H, a = oracle.confidence(x, k)
    for i in range(5):
        top = np.sort(x[i].astype(np.float64))[::-1][:k]
        p = scipy.special.softmax(top)
        np.testing.assert_allclose(a[i], 1.0 - scipy.stats.entropy(p, base=k), rtol=1e-12)
        np.testing.assert_allclose(H[i], scipy.stats.entropy(p), rtol=1e-12)
        # renormalised top-k of the full softmax == softmax of the top-k logits (Eq. 7)
        full = scipy.special.softmax(x[i].astype(np.float64))
        ft = np.sort(full)[::-1][:k]
        np.testing.assert_allclose(ft / ft.sum(), p, rtol=1e-12)


def test_confidence_entropy_bound_given_top_probability():
    k = 10
    x = rng(8).standard_normal((200, 300)).astype(np.float32) * rng(9).uniform(0.2, 6, (200, 1)).astype(np.float32)
    H, a = oracle.confidence(x, k)
    for i in range(200):
        top = np.sort(x[i].astype(np.float64))[::-1][:k]
        p1 = scipy.special.softmax(top)[0]
        assert H[i] <= max_entropy_given_p1(p1, k) + 1e-12
        assert 0.0 <= a[i] <= 1.0
    # The linear bound printed as Lemma 1, p1 >= 1/k + alpha (k-1)/k, is tight at
    # alpha in {0, 1} but is not a valid invariant in between: two equal maxima
    # give alpha = 1 - ln2/ln10 ~ 0.70, so the bound would demand p1 >= 0.73 while p1 = 0.5.
    y = np.full((1, 50), -1e4, np.float32)
    y[0, 4] = y[0, 9] = 0.0
    H, a = oracle.confidence(y, k)
    np.testing.assert_allclose(a[0], 1 - math.log(2) / math.log(10), rtol=1e-12)
    assert 0.5 < 1 / k + a[0] * (k - 1) / k


def test_printed_threshold_value():
    with open(os.path.join(GOLDEN, "acceptance_threshold.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    for k, eps, thr in rows:
        k, eps, thr = int(k), float(eps), float(thr)
        assert round((k - 2 + 4 * eps * k) / (2 * (k - 1)), 2) == thr


# ---------------------------------------------------------------- selection
def test_select_tree_golden_and_monotone():
    with open(os.path.join(GOLDEN, "select_tree_endpoints.txt")) as f:
        rows = [[float(v) for v in ln.split()] for ln in f if ln.strip() and not ln.startswith("#")]
    for a, D, W in rows:
        _, d, w = oracle.select_tree(np.float32([a]), [0.8, 0.4, 0.1])
        assert d[0] == D and w[0] == W
    a = np.linspace(0, 1, 101, dtype=np.float32)
    tid, D, W = oracle.select_tree(a, np.float32([0.8, 0.4, 0.1]))
    assert (np.diff(D) > 0).all() and (np.diff(W) < 0).all() and (np.diff(tid) <= 0).all()
    assert tid[0] == 3 and tid[-1] == 0
    # thresholds are "alpha >= thr keeps the deeper template"
    tid, _, _ = oracle.select_tree(np.float32([0.8, np.nextafter(np.float32(0.8), np.float32(0)), 0.4, 0.1, 0.0999]),
                                   np.float32([0.8, 0.4, 0.1]))
    assert list(tid) == [0, 1, 1, 2, 3]
    tid, _, _ = oracle.select_tree(np.float32([0.5, 0.49, 0.51]), np.float32([0.5]))
    assert list(tid) == [0, 1, 0]


# ---------------------------------------------------------------- expansion
def test_expand_gather_hand_written():
    #      0
    #    1   2        ranks 0,1
    #   3 4  5        3,4 children of 1 (ranks 0,1); 5 child of 2 (rank 0)
    parent = np.array([-1, 0, 0, 1, 1, 2, -1, 0], dtype=np.int32)       # second tree: 2 nodes
    rank = np.array([0, 0, 1, 0, 1, 0, 0, 1], dtype=np.int32)
    offs = np.array([0, 6, 8], dtype=np.int32)
    topk_idx = np.arange(8 * 3).reshape(8, 3) * 10
    got = oracle.expand_gather(topk_idx, parent, rank, offs, np.array([7, 9], dtype=np.int32))
    assert list(got) == [7, 0, 10, 30, 40, 60, 9, 190]


# ---------------------------------------------------------------- acceptance
def best_path_bottom_up(parent, draft, target, max_path):
    """Independent algorithm: mark accepted nodes top-down, then a bottom-up pass
    computes the height of the accepted subtree below every node and follows, from
    the root, the lowest-index child of maximal height."""
    n = len(parent)
    depth = [0] * n
    ok = [False] * n
    ok[0] = True
    for i in range(1, n):
        p = int(parent[i])
        depth[i] = depth[p] + 1
        ok[i] = ok[p] and draft[i] == target[p] and depth[i] < max_path
    height = [1] * n
    choice = [-1] * n
    for i in range(n - 1, 0, -1):
        if ok[i]:
            p = int(parent[i])
            if height[i] + 1 >= height[p]:
                if height[i] + 1 > height[p] or choice[p] < 0 or i < choice[p]:
                    choice[p] = i
                height[p] = height[i] + 1
    out = [0]
    while choice[out[-1]] >= 0:
        out.append(choice[out[-1]])
    return out


def greedy_walk(parent, draft, target):
    """Classic tree verification when sibling tokens are distinct: at most one child matches."""
    n = len(parent)
    out = [0]
    while True:
        nxt = [c for c in range(n) if parent[c] == out[-1] and draft[c] == target[out[-1]]]
        if not nxt:
            return out
        assert len(nxt) == 1
        out.append(nxt[0])


@pytest.mark.parametrize("seed", range(40))
def test_accept_vs_bottom_up_pass(seed):
    r = rng(1000 + seed)
    n = int(r.integers(1, 25))
    t = random_tree(r, n)
    alphabet = int(r.integers(1, 4))            # tiny alphabets: duplicates among siblings, many matches
    draft = r.integers(0, alphabet, n).astype(np.int32)
    target = r.integers(0, alphabet, n).astype(np.int32)
    max_path = int(r.integers(1, 10))
    path, plen, bonus = oracle.accept(t["parent"], draft, target, np.array([0, n], np.int32), max_path)
    want = best_path_bottom_up(t["parent"], draft, target, max_path)
    assert [int(v) for v in path[0, :plen[0]]] == want
    assert (path[0, plen[0]:] == -1).all()
    assert bonus[0] == target[want[-1]]


@pytest.mark.parametrize("seed", range(20))
def test_accept_distinct_siblings_is_the_greedy_walk(seed):
    r = rng(2000 + seed)
    n = int(r.integers(2, 40))
    t = random_tree(r, n)
    # distinct tokens among siblings (what top-k expansion produces): token = 10*rank + small noise class
    draft = (t["rank"] % 3).astype(np.int32) if seed % 2 else t["rank"].astype(np.int32)
    if seed % 2:
        kids = {}
        for i in range(1, n):
            kids.setdefault(int(t["parent"][i]), []).append(i)
        if any(len({int(draft[c]) for c in cs}) != len(cs) for cs in kids.values()):
            draft = t["rank"].astype(np.int32)
    target = r.integers(0, 3, n).astype(np.int32)
    path, plen, bonus = oracle.accept(t["parent"], draft, target, np.array([0, n], np.int32), 64)
    assert [int(v) for v in path[0, :plen[0]]] == greedy_walk(t["parent"], draft, target)


def test_accept_hand_written_cases():
    #        0
    #      1   2          both children carry token 5 (a duplicate among siblings)
    #      |   |
    #      3   4 - 5      1's child carries 9; 2's child 4 carries 7 and 4's child 5 carries 8
    parent = np.array([-1, 0, 0, 1, 2, 4], np.int32)
    draft = np.array([0, 5, 5, 9, 7, 8], np.int32)
    target = np.array([5, 6, 7, 0, 8, 3], np.int32)     # after 1 the target wants 6 (no match); after 2 it wants 7
    path, plen, bonus = oracle.accept(parent, draft, target, np.array([0, 6], np.int32), 8)
    assert [int(v) for v in path[0, :plen[0]]] == [0, 2, 4, 5] and bonus[0] == 3
    # equal lengths: the lower node index wins at the first difference
    target = np.array([5, 9, 7, 0, 1, 3], np.int32)     # [0,1,3] and [0,2,4] both have 3 nodes
    path, plen, bonus = oracle.accept(parent, draft, target, np.array([0, 6], np.int32), 8)
    assert [int(v) for v in path[0, :plen[0]]] == [0, 1, 3] and bonus[0] == 0
    # a match below a mismatch does not count (prefix rule)
    target = np.array([4, 9, 7, 0, 8, 3], np.int32)
    path, plen, bonus = oracle.accept(parent, draft, target, np.array([0, 6], np.int32), 8)
    assert plen[0] == 1 and bonus[0] == 4
    # two trees in one call
    par2 = np.array([-1, 0, 1, -1, 0], np.int32)
    d2 = np.array([0, 3, 4, 0, 8], np.int32)
    t2 = np.array([3, 4, 11, 8, 12], np.int32)
    path, plen, bonus = oracle.accept(par2, d2, t2, np.array([0, 3, 5], np.int32), 4)
    assert plen.tolist() == [3, 2] and bonus.tolist() == [11, 12]
    assert path.tolist() == [[0, 1, 2, -1], [0, 1, -1, -1]]


def test_accept_chain_all_mismatch_and_max_path():
    n = 9
    t = chain_tree(n)
    draft = np.arange(100, 100 + n, dtype=np.int32)
    target = np.array([101, 102, 103, 999, 105, 106, 107, 108, 55], dtype=np.int32)
    path, plen, bonus = oracle.accept(t["parent"], draft, target, np.array([0, n], np.int32), 16)
    assert plen[0] == 4 and list(path[0, :4]) == [0, 1, 2, 3] and bonus[0] == 999   # classic longest prefix
    path, plen, bonus = oracle.accept(t["parent"], draft, np.zeros(n, np.int32), np.array([0, n], np.int32), 16)
    assert plen[0] == 1 and path[0, 0] == 0 and bonus[0] == 0
    full = np.array([101, 102, 103, 104, 105, 106, 107, 108, 55], dtype=np.int32)
    path, plen, bonus = oracle.accept(t["parent"], draft, full, np.array([0, n], np.int32), 16)
    assert plen[0] == 9 and bonus[0] == 55
    path, plen, bonus = oracle.accept(t["parent"], draft, full, np.array([0, n], np.int32), 5)
    assert plen[0] == 5 and bonus[0] == 105                                         # capped by max_path


# ---------------------------------------------------------------- compaction
@pytest.mark.parametrize("path", [[0, 1, 2], [0, 2, 3], [0], [0, 3, 5, 6], [0, 1, 4]])
def test_compact_kv_token_list_model(path):
    r = rng(42)
    L, N, P, Hkv, d, layers = 10, 7, 4, 2, 4, 3
    kv = make_kv_cache(r, [L, 6], [N, 3], [3, 2], Hkv, head_dim=d, page_size=P, n_layers=layers,
                       shuffle=True, spare_frac=0.4)
    # give every (layer, page, head, slot) row a unique content so moves are traceable
    kp = (np.arange(kv["k_pool"].size, dtype=np.uint32) % 65521).astype(np.uint16).reshape(kv["k_pool"].shape)
    vp = ((np.arange(kv["v_pool"].size, dtype=np.uint32) * 7 + 3) % 65521).astype(np.uint16).reshape(kv["v_pool"].shape)
    paths = np.full((2, 8), -1, np.int32)
    paths[0, :len(path)] = path
    second = [0, 1] if path == [0, 1, 2] else [0, 2]
    paths[1, :2] = second
    plen = np.array([len(path), 2], np.int32)
    k2, v2, sl = oracle.compact_kv(kp, vp, kv["page_table"], kv["seq_len"], paths, plen, P)
    assert list(sl) == [L + len(path), 6 + 2]
    # model: per sequence a python list of logical rows; everything else untouched
    for pool, new in ((kp, k2), (vp, v2)):
        want = pool.copy()
        for b, (Lb, pth) in enumerate([(L, path), (6, second)]):
            pt = kv["page_table"][b]
            for layer in range(layers):
                for g in range(Hkv):
                    logical = [pool[layer, pt[t // P], g, t % P].copy() for t in range(Lb + (N if b == 0 else 3))]
                    moved = [logical[Lb + s] for s in pth]
                    for j, row in enumerate(moved):
                        want[layer, pt[(Lb + j) // P], g, (Lb + j) % P] = row
        np.testing.assert_array_equal(new, want)
    if path == [0, 1, 2]:
        np.testing.assert_array_equal(k2, kp)          # identity path: nothing moves


# ---------------------------------------------------------------- generators
def test_templates_have_requested_shape():
    for D, W, N in TEMPLATES + [(8, 2, 60)]:
        t = make_template(D, W, N)
        assert len(t["parent"]) == N and t["parent"][0] == -1
        assert all(0 <= t["parent"][i] < i for i in range(1, N))
        assert t["depth"].max() == D and (np.diff(t["depth"]) >= 0).all()
        kids = np.bincount(t["parent"][1:], minlength=N)
        assert kids.max() <= W
        for p in range(N):
            rk = sorted(t["rank"][i] for i in range(1, N) if t["parent"][i] == p)
            assert len(set(rk)) == len(rk) and all(0 <= v < W for v in rk)


def test_bf16_round_trip():
    x = rng(0).standard_normal(1000).astype(np.float32)
    b = bf16_bits(x)
    y = bf16_to_f32(b)
    assert np.abs(y - x).max() <= np.abs(x).max() * 2.0 ** -8
    np.testing.assert_array_equal(bf16_bits(y), b)
    assert bf16_bits(np.float32([1.00390625]))[0] == 0x3F80      # tie -> even
    assert bf16_bits(np.float32([1.01171875]))[0] == 0x3F82      # tie -> even (up)
