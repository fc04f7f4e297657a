"""Draft-side tree attention (Section 3.3 "Phase 1": the draft model fills the tree level by level;
Section 5.1: 80 to 90 % of the visual tokens are pruned for the draft, so its cache is a tenth to a
fifth of the target's).  The same sage_tree_attention call serves that regime: short context, a tree
that grows by one level per call (1 ... W new nodes), queries for every node so far.  After every
level of sage_grow_tree the attention over the tree built so far is compared with the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_00523_b200 as sage
from helpers import check_attention, dev_bf16, dev_f32, dev_i32, host_bits
from workloads import make_kv_cache, make_q

pytestmark = pytest.mark.gpu

CAP, K = sage.SAGE_MAX_NODES, 8
HQ, HKV, D, P = 64, 8, 128, 64


@pytest.mark.parametrize("target_len,pruned", [(4096, 0.9), (16384, 0.8)])
def test_attention_over_a_tree_that_grows_level_by_level_in_the_pruned_draft_cache(target_len, pruned):
    rng = np.random.Generator(np.random.Philox(int(target_len * pruned)))
    n_visual = int(0.75 * target_len)
    L = target_len - int(pruned * n_visual)                  # what is left of the context for the draft model
    kv = make_kv_cache(rng, [L], [CAP], [n_visual - int(pruned * n_visual)], HKV, shuffle=True, spare_frac=0.2)
    q = make_q(rng, CAP, HQ, D)
    # candidate rows of every node slot: a clear first choice and plausible alternatives
    lp = np.zeros((CAP, K), np.float32)
    for r in range(CAP):
        p = np.sort(rng.dirichlet(np.ones(K) * 0.4))[::-1]
        lp[r] = np.log(np.maximum(p, 1e-30))
    ix = rng.integers(0, 150000, size=(CAP, K)).astype(np.int32)
    alpha = np.float32([0.35])
    host = dict(parent=np.full(CAP, -1, np.int32), rank=np.zeros(CAP, np.int32), depth=np.zeros(CAP, np.int32),
                token=np.zeros(CAP, np.int32), cum_logprob=np.zeros(CAP, np.float32))
    n, fb = 1, 0
    tree = {name: (dev_f32(a) if a.dtype == np.float32 else dev_i32(a)) for name, a in host.items()}
    tree["n_nodes"], tree["frontier_begin"] = dev_i32([1]), dev_i32([0])
    pol = sage.make_policy([])
    k_d, v_d, q_d = dev_bf16(kv["k_pool"]), dev_bf16(kv["v_pool"]), dev_bf16(q)
    pt_d, sl_d = dev_i32(kv["page_table"]), dev_i32(kv["seq_len"])
    st = sage.new_status()
    sizes = []
    for level in range(8):
        sage.sage_grow_tree(dev_i32(ix), dev_f32(lp), dev_f32(alpha), pol, tree, status=st)
        n, fb = oracle.grow_tree_level(host["parent"], host["rank"], host["depth"], host["token"], host["cum_logprob"],
                                       n, fb, ix, lp, alpha[0])
        assert int(tree["n_nodes"].item()) == n
        np.testing.assert_array_equal(tree["parent"].cpu().numpy()[:n], host["parent"][:n])
        sizes.append(n)
        offs = np.array([0, n], np.int32)
        out = sage.sage_tree_attention(q_d, k_d, v_d, pt_d, sl_d, tree["parent"], dev_i32(offs), 1.0 / np.sqrt(D), status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0, sage.status_string(int(st.item()))
        want = oracle.tree_attention(q[0], kv["k_pool"][0], kv["v_pool"][0], kv["page_table"], kv["seq_len"],
                                     host["parent"][:n], offs, HQ, HKV, D, P, 1.0 / np.sqrt(D))
        check_attention(host_bits(out)[0][:n], want[:n])
    assert sizes[0] >= 2 and sizes[-1] > sizes[0] and sizes[-1] <= CAP      # the tree really grew over the calls
