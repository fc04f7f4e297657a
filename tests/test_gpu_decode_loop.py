"""The device decode loop (paper_2602_00523_b200.decode_loop: Algorithm 1 with synthetic model
stand-ins, no host round trip between rounds) against the CPU reference loop built from the oracle,
round by round and bit for bit: tree shapes, draft tokens, accepted paths, tau + 1, bonus tokens,
template ids, the history controller's maximum depth, sequence lengths and the final compacted cache.
Four policies at the same node budget: SD-Chain, a static SD-Tree, entropy-selected templates
(look-ahead), and trees grown level by level with the depth steered by the acceptance history.
For the chain policy the mean acceptance length over many rounds is also held against the closed form
of the expected-acceptance theorem (Section 4.2)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_00523_b200 as sage
from paper_2602_00523_b200.decode_loop import DecodeLoop, SyntheticTarget
from helpers import dev_bf16, dev_f32, dev_i32, host_bits
from loop_reference import reference_loop
from workloads import TEMPLATES, acceptance_picks, chain_tree, make_kv_cache, make_loop_logits, make_q, make_template

pytestmark = pytest.mark.gpu

HQ, HKV, D, P = 16, 2, 128, 64
K, KE, MAX_PATH, CAP = 10, 10, 9, 64
BUDGET = 40


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def build(policy, rounds, seed, vocab, prefix, kinds, p_acc, gamma, layers=1, trees=None, thresholds=(), tree_kw=None):
    r = rng(seed)
    draft = [make_loop_logits(r, CAP, vocab, kd) for kd in kinds]
    picks = acceptance_picks(r, rounds, CAP, 8, K, p_acc, gamma)
    noise = r.standard_normal((CAP, vocab), dtype=np.float32)
    kv = make_kv_cache(r, [prefix], [CAP + rounds * MAX_PATH], [prefix // 2], HKV, n_layers=layers, shuffle=True,
                       spare_frac=0.2, poison=False)
    q = make_q(r, CAP, HQ, D, layers)
    loop = DecodeLoop(policy=policy, draft_logits=[dev_f32(d) for d in draft], target=SyntheticTarget(dev_f32(noise), picks, K),
                      k=K, k_entropy=KE, q=dev_bf16(q), k_pool=dev_bf16(kv["k_pool"]), v_pool=dev_bf16(kv["v_pool"]),
                      page_table=dev_i32(kv["page_table"]), prefix_len=prefix, max_path=MAX_PATH, trees=trees,
                      thresholds=thresholds, n_budget=BUDGET, tree_policy_kw=tree_kw, rounds_capacity=rounds)
    return loop, draft, picks, kv


POLICIES = {
    "chain": dict(trees=[chain_tree(9)]),
    "static": dict(trees=[make_template(4, 6, BUDGET)]),
    "templates": dict(trees=[make_template(d, w, BUDGET) for d, w, _ in TEMPLATES], thresholds=[0.8, 0.4, 0.1]),
    "dynamic": dict(tree_kw=dict(d_min=3.0, d_max=6.0, w_min=2.0, w_max=10.0)),
}


@pytest.mark.parametrize("policy", ["chain", "static", "templates", "dynamic"])
def test_device_loop_matches_the_reference_loop_round_by_round(policy):
    rounds, vocab, prefix = 30, 8192, 500
    kinds = ["low", "high", "steps:5.5", "mid:3.0", "steps:4", "low", "mid:1.8", "steps:7", "high"]
    cfg = POLICIES[policy]
    loop, draft, picks, kv = build(policy, rounds, 900 + len(policy), vocab, prefix, kinds, 0.85, 0.95, layers=2,
                                   trees=cfg.get("trees"), thresholds=cfg.get("thresholds", ()), tree_kw=cfg.get("tree_kw"))
    rec = {n: t.cpu().numpy() for n, t in loop.run(rounds).items()}
    torch.cuda.synchronize()
    assert int(loop.status.item()) == 0, sage.status_string(int(loop.status.item()))
    ref = reference_loop(policy, rounds, draft, picks, K, KE, MAX_PATH, trees=cfg.get("trees"),
                         thresholds=cfg.get("thresholds", ()), n_budget=BUDGET, tree_policy_kw=cfg.get("tree_kw"),
                         kv=dict(k_pool=kv["k_pool"], v_pool=kv["v_pool"], page_table=kv["page_table"],
                                 seq_len=kv["seq_len"]))
    want = ref["rec"]
    for name in ("path_len", "n_nodes", "bonus", "seq_len"):
        np.testing.assert_array_equal(rec[name][:rounds], np.array(want[name]), err_msg=name)
    np.testing.assert_array_equal(rec["d_max"][:rounds], np.array(want["d_max"], np.float32))
    assert np.abs(rec["alpha"][:rounds] - np.array(want["alpha"])).max() <= 1e-5
    if policy == "templates":
        np.testing.assert_array_equal(rec["template"][:rounds], np.array(want["template"]))
        assert len(set(want["template"])) >= 3                 # the loop really moved between templates
    for r in range(rounds):
        n = want["n_nodes"][r]
        np.testing.assert_array_equal(rec["tree_parent"][r][:n], want["tree_parent"][r][:n], err_msg=f"round {r}")
        np.testing.assert_array_equal(rec["draft_token"][r][:n], want["draft_token"][r][:n], err_msg=f"round {r}")
        np.testing.assert_array_equal(rec["path"][r], want["path"][r], err_msg=f"round {r}")
    assert max(want["path_len"]) > 2 and min(want["path_len"]) >= 1
    if policy == "dynamic":
        assert len(set(want["n_nodes"])) > 3 and max(want["n_nodes"]) <= BUDGET
    # the cache after all rounds: every accepted row moved exactly as in the oracle's chain of compactions
    assert np.array_equal(host_bits(loop.k_pool), ref["k_pool"])
    assert np.array_equal(host_bits(loop.v_pool), ref["v_pool"])


def test_chain_policy_on_the_device_reaches_the_closed_form_mean_acceptance_length():
    p_acc, gamma, depth, rounds = 0.8, 0.9, 6, 3000
    loop, _, _, _ = build("chain", rounds, 77, 2048, 64, ["mixed", "low", "high"], p_acc, gamma, trees=[chain_tree(depth + 1)])
    rec = loop.run(rounds)
    torch.cuda.synchronize()
    assert int(loop.status.item()) == 0
    tau = rec["path_len"].cpu().numpy()[:rounds].astype(np.float64) - 1
    want = oracle.expected_acceptance_length(p_acc, gamma, depth)
    se = tau.std() / np.sqrt(rounds)
    assert abs(tau.mean() - want) < 4 * se, (tau.mean(), want, se)
