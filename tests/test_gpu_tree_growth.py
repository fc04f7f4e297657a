"""GPU parity of sage_grow_tree against the oracle's level-by-level construction: bit-exact
parent / rank / depth / token arrays, node counts and frontiers, and identical fp32 cumulative
log-probabilities, level after level, for a batch of sequences with different confidences."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_00523_b200 as sage
from helpers import dev_f32, dev_i32

pytestmark = pytest.mark.gpu

CAP = sage.SAGE_MAX_NODES


def candidate_rows(rng, k, sharp):
    """Descending log-probabilities of one node's k candidates (a stand-in for the draft model)."""
    p = np.sort(rng.dirichlet(np.ones(k + 4) * sharp))[::-1][:k]
    return np.log(np.maximum(p, 1e-30)).astype(np.float32)


def run_case(seed, alphas, k, n_max, policy_kw, sharp):
    rng = np.random.Generator(np.random.Philox(seed))
    B = len(alphas)
    lp = np.zeros((B * CAP, k), np.float32)
    ix = np.zeros((B * CAP, k), np.int32)
    for row in range(B * CAP):                     # every slot gets a row up front: slots are reused by index only
        lp[row] = sharp(rng, k) if callable(sharp) else candidate_rows(rng, k, sharp)
        ix[row] = rng.choice(150000, size=k, replace=False)
    host = dict(parent=np.full(B * CAP, -1, np.int32), rank=np.zeros(B * CAP, np.int32),
                depth=np.zeros(B * CAP, np.int32), token=np.zeros(B * CAP, np.int32),
                cum_logprob=np.zeros(B * CAP, np.float32))
    n_nodes = np.ones(B, np.int32)
    frontier = np.zeros(B, np.int32)
    for b in range(B):
        host["token"][b * CAP] = 7 + b
    tree = {name: (dev_f32(a) if a.dtype == np.float32 else dev_i32(a)) for name, a in host.items()}
    tree["n_nodes"], tree["frontier_begin"] = dev_i32(n_nodes), dev_i32(frontier)
    pol = sage.make_policy([], **policy_kw)
    d_lp, d_ix, d_alpha = dev_f32(lp), dev_i32(ix), dev_f32(np.asarray(alphas, np.float32))
    st = sage.new_status()
    total_levels = 0
    for level in range(12):
        sage.sage_grow_tree(d_ix, d_lp, d_alpha, pol, tree, n_max=n_max, status=st)
        for b in range(B):
            sl = slice(b * CAP, (b + 1) * CAP)
            n2, f2 = oracle.grow_tree_level(host["parent"][sl], host["rank"][sl], host["depth"][sl],
                                            host["token"][sl], host["cum_logprob"][sl], n_nodes[b], frontier[b],
                                            ix[sl], lp[sl], alphas[b], n_max=n_max, **policy_kw)
            total_levels += int(n2 > n_nodes[b])
            n_nodes[b], frontier[b] = n2, f2
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        np.testing.assert_array_equal(tree["n_nodes"].cpu().numpy(), n_nodes)
        np.testing.assert_array_equal(tree["frontier_begin"].cpu().numpy(), frontier)
        for name in ("parent", "rank", "depth", "token"):
            np.testing.assert_array_equal(tree[name].cpu().numpy(), host[name], err_msg=name)
        np.testing.assert_array_equal(tree["cum_logprob"].cpu().numpy().view(np.uint32),
                                      host["cum_logprob"].view(np.uint32))
    return n_nodes, total_levels


def test_grow_tree_paper_policy_batch_of_confidences():
    alphas = [0.0, 0.02, 0.25, 0.5, 0.77, 0.93, 1.0, 0.5]
    n_nodes, levels = run_case(11, alphas, k=10, n_max=64, policy_kw=dict(d_min=3.0, d_max=8.0, w_min=2.0, w_max=10.0),
                               sharp=0.3)
    assert levels > len(alphas)                       # trees really grew over several levels
    assert n_nodes.max() <= 64 and n_nodes.min() >= 2


def test_grow_tree_hits_the_node_budget_and_small_k():
    def four_strong(rng, k):
        # four candidates near 0.24 each, the rest tiny: three levels of a wide tree overflow 64 nodes
        p = np.concatenate([0.24 - 0.01 * np.sort(rng.random(4)), np.full(k - 4, 1e-4)])
        return np.log(p).astype(np.float32)
    n_nodes, _ = run_case(12, [0.0, 0.1, 0.0], k=16, n_max=64,
                          policy_kw=dict(d_min=64.0, d_max=64.0, w_min=2.0, w_max=16.0), sharp=four_strong)
    assert n_nodes.max() == 64                        # the node budget cut the third level short
    run_case(13, [0.3, 0.9], k=1, n_max=9, policy_kw=dict(d_min=2.0, d_max=12.0, w_min=1.0, w_max=1.0), sharp=0.05)


def test_grow_tree_rejects_bad_state():
    tree = dict(parent=dev_i32(np.full(CAP, -1)), rank=dev_i32(np.zeros(CAP)), depth=dev_i32(np.zeros(CAP)),
                token=dev_i32(np.zeros(CAP)), cum_logprob=dev_f32(np.zeros(CAP)),
                n_nodes=dev_i32([70]), frontier_begin=dev_i32([0]))
    st = sage.new_status()
    sage.sage_grow_tree(dev_i32(np.zeros((CAP, 4))), dev_f32(np.zeros((CAP, 4))), dev_f32([0.5]), sage.make_policy([]),
                        tree, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == sage.SAGE_STATUS_BAD_TREE
