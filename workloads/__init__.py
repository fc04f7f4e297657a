"""Seeded synthetic inputs for the SAGE decode-round hot path.

This package only *draws data*: random tensors, page tables, tree shapes and
planted logits.  It holds none of the method's arithmetic (no softmax, no
top-k, no attention, no acceptance walk), so that the CPU oracle and the CUDA
path can both consume exactly the same bytes without sharing any code that
computes a result.
"""
from .gen import (  # noqa: F401
    bf16_bits, bf16_to_f32, make_template, random_tree, chain_tree, star_tree,
    make_kv_cache, make_q, place_rows, make_logits, make_target_logits, make_config,
    markov_entropy_states, TEMPLATES, CONFIG_NAMES, seed_for,
    acceptance_picks, make_loop_logits, NO_CANDIDATE,
)
