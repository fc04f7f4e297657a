"""CPU oracle for the SAGE decode-round hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 NumPy statement of what each step of the path computes,
written from the paper's definitions.  It exists to check the CUDA library and
to serve as the timed CPU baseline of the benchmark; it is not a fallback.
Only the tests, the smoke check and the benchmark's CPU-baseline / reference
legs may import it.  It shares no code with the CUDA path and imports nothing
from it.

Pin status (what fixes each function other than itself, see tests/test_oracle_*):
  ancestor_mask      brute-force parent-chain walk; chain / star closed forms
  tree_attention     brute-force dense masked attention in pure Python loops,
                     chain tree == causal attention, non-ancestor perturbation,
                     page permutation, equal-keys mean, single-node decode
  softmax_entropy    ln V (constant row), 0 (one-hot), two-level closed form
  topk               full sort on tiny rows, planted ties, constant row
  confidence         alpha = 0 (uniform top-k), alpha -> 1 (one dominant),
                     log-base independence, max-entropy bound given p_1
  select_tree        D(0)=3, D(1)=8, W(0)=10, W(1)=2, alpha=0.5 -> (5.5, 6)
  expand_gather      direct definition on hand-written trees
  accept             exhaustive enumeration of root-to-leaf paths
  compact_kv         whole-pool byte comparison against a token-list model
  grow_tree_level    the path-inclusion rule evaluated directly on every path of a full
                     k-ary tree (tiny k, depth); its readings of the paper's rounding /
                     P_parent / stopping order are "parity unpinned"
  update_history     hand-computed windows; its long-run behaviour under a simulated
                     acceptance process whose mean is the closed form of Theorem 2
                     (expected_acceptance_length, itself checked by simulation); step, clamps
                     and the warm-up rule are "parity unpinned"
  Which row of a tree supplies the distribution that drives selection is not
  fixed by the paper: "parity unpinned" for that choice (the caller passes the
  row index to both sides).
"""
from .sage_oracle import (  # noqa: F401
    ancestor_mask, tree_attention, softmax_entropy, topk, topk_logprob,
    confidence, select_tree, expand_gather, accept, compact_kv, widen_bf16, grow_tree_level, update_history, expected_acceptance_length,
)
