"""Pins for the oracle's adaptive history tracking (Section 3.3) and for the closed-form expected
acceptance length (Theorem 2, Section 4.2) that drives its long-run test."""
import numpy as np

import oracle


def simulate_tau(rng, p, gamma, depth):
    """Greedy-path speculation: the level-l token is accepted with probability p gamma^(l-1); tau is the
    number of accepted levels before the first rejection."""
    tau = 0
    for l in range(1, depth + 1):
        if rng.random() < p * gamma ** (l - 1):
            tau += 1
        else:
            break
    return tau


def test_expected_acceptance_length_matches_simulation_and_textbook_cases():
    # gamma = 1: geometric series p (1 - p^D) / (1 - p)
    for p, D in [(0.5, 4), (0.9, 8), (0.2, 3)]:
        assert abs(oracle.expected_acceptance_length(p, 1.0, D) - p * (1 - p ** D) / (1 - p)) < 1e-12
    assert oracle.expected_acceptance_length(1.0, 1.0, 8) == 8.0
    rng = np.random.Generator(np.random.Philox(77))
    for p, g, D in [(0.8, 0.9, 6), (0.6, 1.0, 8), (0.95, 0.8, 5)]:
        sims = np.mean([simulate_tau(rng, p, g, D) for _ in range(40000)])
        assert abs(sims - oracle.expected_acceptance_length(p, g, D)) < 0.03


def test_update_history_hand_computed_window():
    buf = np.zeros(4, np.int32)
    count, d = 0, np.float32(5.0)
    kw = dict(window=4, lower=2.0, upper=3.0, step=1.0, d_lo=3.0, d_hi=8.0, min_samples=4)
    seq = [1, 1, 1, 1, 4, 4, 4, 4, 4, 2, 3, 2, 3]
    got = []
    for tau in seq:
        count, d = oracle.update_history(buf, count, d, tau, **kw)
        got.append(float(d))
    # by hand: three warm-up samples hold 5; {1,1,1,1} mean 1 -> 4; {1,1,1,4} mean 1.75 -> 3;
    # {1,1,4,4} mean 2.5 holds; {1,4,4,4} mean 3.25 -> 4; {4,4,4,4} -> 5; {4,4,4,4} -> 6;
    # {4,4,4,2} mean 3.5 -> 7; {4,4,2,3} mean 3.25 -> 8; {4,2,3,2} mean 2.75 holds; {2,3,2,3} holds
    assert got == [5, 5, 5, 4, 3, 3, 4, 5, 6, 7, 8, 8, 8]
    # and once more from the definition, without a ring buffer
    exp, dd = [], 5.0
    for i in range(len(seq)):
        if i + 1 >= 4:
            mean = sum(seq[i - 3:i + 1]) / 4.0
            if mean < 2.0:
                dd = max(3.0, dd - 1.0)
            elif mean > 3.0:
                dd = min(8.0, dd + 1.0)
        exp.append(dd)
    assert got == exp


def test_update_history_long_run_follows_the_expected_acceptance_length():
    rng = np.random.Generator(np.random.Philox(5))
    for p, target in [(0.95, 8.0), (0.35, 3.0)]:
        # E[tau] at depth 8 with gamma = 1: 6.4 for p = 0.95 (> 3: depth climbs), 0.54 for p = 0.35 (< 2: falls)
        assert (oracle.expected_acceptance_length(p, 1.0, 8) > 3.0) == (target == 8.0)
        buf = np.zeros(10, np.int32)
        count, d = 0, np.float32(5.0)
        for _ in range(200):
            tau = simulate_tau(rng, p, 1.0, int(d))
            count, d = oracle.update_history(buf, count, d, tau)
        assert float(d) == target


def test_update_history_holds_between_the_thresholds():
    buf = np.zeros(10, np.int32)
    count, d = 0, np.float32(6.0)
    for i in range(50):
        count, d = oracle.update_history(buf, count, d, 2 + (i % 2))       # mean 2.5
    assert float(d) == 6.0
