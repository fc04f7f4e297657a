"""CPU pins of the reference decode loop (tests/loop_reference.py), which the device loop is compared
with: under the synthetic acceptance process a chain of depth D is accepted level by level with
probability p * gamma^(l-1), so the mean acceptance length over many rounds must be the closed form of
the expected-acceptance theorem (Section 4.2), sum_l p^l gamma^(l(l-1)/2); a wider tree of the same
depth accepts more on average; and the history controller must steer the maximum depth."""
import numpy as np

import oracle
from loop_reference import reference_loop
from workloads import acceptance_picks, chain_tree, make_loop_logits, make_template


def rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def small_logits(seed, n_buffers=4, vocab=128, kind="mixed"):
    r = rng(seed)
    return [make_loop_logits(r, 64, vocab, kind) for _ in range(n_buffers)]


def test_chain_policy_mean_acceptance_matches_the_closed_form():
    p, gamma, depth, rounds = 0.8, 0.9, 6, 3000
    picks = acceptance_picks(rng(1), rounds, 64, 8, 4, p, gamma)
    out = reference_loop("chain", rounds, small_logits(2), picks, k=4, k_entropy=4, max_path=9, trees=[chain_tree(depth + 1)])
    tau = np.array(out["rec"]["path_len"]) - 1
    want = oracle.expected_acceptance_length(p, gamma, depth)
    se = tau.std() / np.sqrt(rounds)
    assert abs(tau.mean() - want) < 4 * se + 1e-9, (tau.mean(), want, se)
    assert tau.max() == depth and tau.min() == 0


def test_a_wider_tree_of_the_same_depth_accepts_at_least_as_much_as_the_chain():
    p, gamma, rounds = 0.6, 0.9, 1500
    picks = acceptance_picks(rng(3), rounds, 64, 8, 4, p, gamma)
    lg = small_logits(4)
    chain = reference_loop("chain", rounds, lg, picks, k=4, k_entropy=4, max_path=9, trees=[chain_tree(5)])
    wide = reference_loop("static", rounds, lg, picks, k=4, k_entropy=4, max_path=9, trees=[make_template(4, 3, 30)])
    a, b = np.array(chain["rec"]["path_len"]), np.array(wide["rec"]["path_len"])
    # the tree contains a chain of the same depth and catches the target's second and third choices too
    assert b.mean() > a.mean() + 0.3
    assert a.max() <= 5 and b.max() <= 5


def test_history_controller_moves_the_depth_in_the_dynamic_policy():
    rounds = 120
    lg = small_logits(5, kind="low")          # confident draft: deep, narrow trees
    good = reference_loop("dynamic", rounds, lg, acceptance_picks(rng(6), rounds, 64, 8, 4, 0.97, 1.0), k=4, k_entropy=4,
                          max_path=9, tree_policy_kw=dict(d_max=5.0))
    bad = reference_loop("dynamic", rounds, lg, acceptance_picks(rng(7), rounds, 64, 8, 4, 0.15, 1.0), k=4, k_entropy=4,
                         max_path=9, tree_policy_kw=dict(d_max=5.0))
    assert good["rec"]["d_max"][-1] == 8.0 and bad["rec"]["d_max"][-1] == 3.0
    assert max(good["rec"]["n_nodes"]) <= 64 and min(good["rec"]["n_nodes"]) >= 1
