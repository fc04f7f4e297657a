"""Shared test plumbing: host<->device conversion and the oracle-side round."""
import numpy as np
import torch

import oracle
from workloads import make_target_logits
from workloads.gen import _rng

# Attention tolerance.  Target: max |a-b| <= 1e-2 and, per (node, head) row,
# max|a-b| / max|b| <= 1e-2.  The output is stored in bf16, whose rounding alone is up to
# 2^-8 |b| (0.0156 at |b| = 4), so the absolute bound is scaled by max(1, row max |b|):
# it is exactly 1e-2 wherever outputs stay below 1 in magnitude (all long-context rows).
ATTN_MAX_ABS = 1e-2
ATTN_ROW_REL = 1e-2
ENTROPY_ABS = 1e-5


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def dev_i32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def dev_f32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def widen(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def check_attention(got_bits: np.ndarray, want: np.ndarray):
    """got: bf16 bits [nodes, Hq, d]; want: fp64 same shape."""
    got = widen(got_bits)
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    row_mag = np.abs(want).max(axis=-1)
    excess = err.max(axis=-1) / np.maximum(1.0, row_mag)
    assert excess.max() <= ATTN_MAX_ABS, f"max abs err {err.max()} (scaled {excess.max()})"
    row_rel = err.max(axis=-1) / row_mag
    assert row_rel.max() <= ATTN_ROW_REL, f"max row-relative err {row_rel.max()}"
    return float(err.max()), float(row_rel.max())


def oracle_attention_layer(c, layer):
    return oracle.tree_attention(c["q"][layer], c["k_pool"][layer], c["v_pool"][layer], c["page_table"],
                                 c["seq_len"], c["parent"], c["node_offsets"], c["n_q_heads"], c["n_kv_heads"],
                                 c["head_dim"], c["page_size"], c["sm_scale"])


def oracle_logits_side(c, rnd=0):
    """Oracle results for the draft logits of one round."""
    lg = c["draft_logits"][rnd]
    H, lse = oracle.softmax_entropy(lg)
    idx = oracle.topk(lg, c["k"])
    Ht, alpha = oracle.confidence(lg, c["k_entropy"])
    lp = oracle.topk_logprob(lg, idx, lse)
    tok = oracle.expand_gather(idx, c["parent"], c["rank"], c["node_offsets"], c["root_token"])
    return {"entropy_full": H, "lse": lse, "topk_idx": idx, "entropy_topk": Ht, "alpha": alpha,
            "topk_logprob": lp, "draft_token": tok}


def target_logits_for(c, draft_token, tensor_id=7):
    """Target logits for every tree of the config with a planted accepted path
    (towards a seeded node of each tree).  draft_token comes from the oracle."""
    r = _rng(c["cfg"], tensor_id)
    rows, accept_nodes = [], []
    for b, t in enumerate(c["trees"]):
        n0, n1 = int(c["node_offsets"][b]), int(c["node_offsets"][b + 1])
        node = int(r.integers(0, n1 - n0))
        accept_nodes.append(node)
        rows.append(make_target_logits(r, t, draft_token[n0:n1], node, c["vocab"])["logits"])
    return np.concatenate(rows, axis=0), accept_nodes
