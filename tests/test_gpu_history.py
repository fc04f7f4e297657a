"""GPU parity of sage_update_history against the oracle (bit-exact window contents, counts and
maximum depths over a long run of a batch of sequences), and of sage_grow_tree with the
per-sequence maximum depth that the controller produces."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_00523_b200 as sage
from helpers import dev_f32, dev_i32

pytestmark = pytest.mark.gpu


def test_update_history_matches_oracle_over_many_rounds():
    rng = np.random.Generator(np.random.Philox(31))
    B, W = 16, 10
    pol_kw = dict(window=W, lower=2.0, upper=3.0, step=1.0, d_lo=3.0, d_hi=8.0, min_samples=W)
    pol = sage.make_history_policy(**pol_kw)
    buf_h = np.zeros((B, W), np.int32); cnt_h = np.zeros(B, np.int32); d_h = np.full(B, 5.0, np.float32)
    buf_d, cnt_d, d_d = dev_i32(buf_h), dev_i32(cnt_h), dev_f32(d_h)
    p_accept = rng.uniform(0.2, 0.97, size=B)            # per-sequence draft quality
    st = sage.new_status()
    for rnd in range(120):
        tau = np.array([min(int(rng.geometric(1 - p)) - 1, int(d)) for p, d in zip(p_accept, d_h)], np.int32)
        sage.sage_update_history(dev_i32(tau + 1), pol, buf_d, cnt_d, d_d, status=st)
        for b in range(B):
            cnt_h[b], d_h[b] = oracle.update_history(buf_h[b], cnt_h[b], d_h[b], tau[b], **pol_kw)
        if rnd % 10 == 9:
            torch.cuda.synchronize()
            np.testing.assert_array_equal(buf_d.cpu().numpy(), buf_h)
            np.testing.assert_array_equal(cnt_d.cpu().numpy(), cnt_h)
            np.testing.assert_array_equal(d_d.cpu().numpy().view(np.uint32), d_h.view(np.uint32))
    assert int(st.item()) == 0
    assert d_h.min() == 3.0 and d_h.max() == 8.0         # both ends of the clamp were reached


def test_update_history_rejects_an_empty_path():
    pol = sage.make_history_policy()
    st = sage.new_status()
    sage.sage_update_history(dev_i32([0]), pol, dev_i32(np.zeros((1, 10))), dev_i32([0]), dev_f32([5.0]), status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == sage.SAGE_STATUS_BAD_PATH


def test_grow_tree_with_per_sequence_maximum_depth():
    rng = np.random.Generator(np.random.Philox(32))
    CAP, k, B = sage.SAGE_MAX_NODES, 6, 4
    d_max_seq = np.array([3.0, 5.0, 8.0, 6.0], np.float32)
    alphas = np.array([1.0, 1.0, 1.0, 0.5], np.float32)
    lp = np.zeros((B * CAP, k), np.float32)
    for r in range(B * CAP):
        p = np.sort(rng.dirichlet(np.ones(k) * 0.2))[::-1]
        lp[r] = np.log(np.maximum(p, 1e-30))
    ix = rng.integers(0, 150000, size=(B * CAP, k)).astype(np.int32)
    host = dict(parent=np.full(B * CAP, -1, np.int32), rank=np.zeros(B * CAP, np.int32), depth=np.zeros(B * CAP, np.int32),
                token=np.zeros(B * CAP, np.int32), cum_logprob=np.zeros(B * CAP, np.float32))
    n_nodes, frontier = np.ones(B, np.int32), np.zeros(B, np.int32)
    tree = {n: (dev_f32(a) if a.dtype == np.float32 else dev_i32(a)) for n, a in host.items()}
    tree["n_nodes"], tree["frontier_begin"] = dev_i32(n_nodes), dev_i32(frontier)
    pol = sage.make_policy([])
    st = sage.new_status()
    for _ in range(10):
        sage.sage_grow_tree(dev_i32(ix), dev_f32(lp), dev_f32(alphas), pol, tree, d_max_seq=dev_f32(d_max_seq), status=st)
        for b in range(B):
            sl = slice(b * CAP, (b + 1) * CAP)
            n_nodes[b], frontier[b] = oracle.grow_tree_level(host["parent"][sl], host["rank"][sl], host["depth"][sl],
                                                             host["token"][sl], host["cum_logprob"][sl], n_nodes[b],
                                                             frontier[b], ix[sl], lp[sl], alphas[b],
                                                             d_max=float(d_max_seq[b]))
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    np.testing.assert_array_equal(tree["n_nodes"].cpu().numpy(), n_nodes)
    np.testing.assert_array_equal(tree["frontier_begin"].cpu().numpy(), frontier)
    for name in ("parent", "rank", "depth", "token"):
        np.testing.assert_array_equal(tree[name].cpu().numpy(), host[name])
    np.testing.assert_array_equal(tree["cum_logprob"].cpu().numpy().view(np.uint32), host["cum_logprob"].view(np.uint32))
    depth_reached = [int(host["depth"][b * CAP:b * CAP + n_nodes[b]].max()) for b in range(B)]
    assert depth_reached[0] <= 3 and depth_reached[1] <= 5 and depth_reached[0] < depth_reached[2]
