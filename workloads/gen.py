"""Seeded input generators for the five workload configurations.

Everything here is data: Gaussian tensors rounded to bf16, page tables,
speculation-tree shapes (parent / rank arrays) and logits rows with planted
peaks.  Both the CPU oracle and the CUDA library are fed the arrays made here,
byte for byte.  Nothing in this file computes a softmax, a top-k, an attention
output or an acceptance path.

Seeds: ``seed = 523000 + 1000 * config + tensor_id`` drives a Philox generator
(``numpy.random.Philox``), so every tensor of every configuration can be
re-drawn independently.

Workload shapes follow the Qwen2.5-VL-72B decoder layer (64 query heads, 8 KV
heads, head_dim 128, vocabulary 152064, 80 layers) and the paper's tree
hyper-parameters (depth 3..8, width 2..10, at most 64 nodes; Section 5.1,
"Implementation details").
"""
from __future__ import annotations

import heapq
from typing import Dict, List, Optional, Sequence

import numpy as np

# (depth, width, nodes incl. root) -- ordered from the most confident template
# (deep / narrow) to the least confident one (shallow / wide).
TEMPLATES = [(8, 2, 24), (6, 3, 36), (4, 6, 48), (3, 10, 60)]

CONFIG_NAMES = {
    1: "tiny-single-group",
    2: "qwen72b-2k-deep-narrow",
    3: "qwen72b-4k-shallow-wide",
    4: "qwen72b-16k-video",
    5: "qwen72b-batch16-ragged",
}

POISON_BF16 = np.uint16(0x7FC0)  # bf16 quiet NaN: fills cache rows nobody may read


def seed_for(config: int, tensor_id: int) -> int:
    return 523000 + 1000 * int(config) + int(tensor_id)


def _rng(config: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(seed_for(config, tensor_id)))


# --------------------------------------------------------------------------
# bf16 <-> fp32 bit conversions (storage format only)
# --------------------------------------------------------------------------
def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round finite fp32 values to bf16 (round-to-nearest-even); returns uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 exactly."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# Trees.  A tree is data for every kernel: parent[i] < i, parent[0] = -1,
# rank[i] = which of its parent's top-k candidates node i carries.
# --------------------------------------------------------------------------
def _finish_tree(parent: Sequence[int], rank: Sequence[int]) -> Dict[str, np.ndarray]:
    parent = np.asarray(parent, dtype=np.int32)
    rank = np.asarray(rank, dtype=np.int32)
    depth = np.zeros(len(parent), dtype=np.int32)
    for i in range(1, len(parent)):
        depth[i] = depth[parent[i]] + 1
    return {"parent": parent, "rank": rank, "depth": depth}


def make_template(depth: int, width: int, n_nodes: int, decay: float = 0.6) -> Dict[str, np.ndarray]:
    """Deterministic (depth, width, n_nodes) tree shape.

    Candidates are the nodes of the full ``width``-ary tree of the given depth.
    The child of rank j gets conditional weight proportional to ``decay**j``; a
    candidate's score is the product of the weights along its path.  The rank-0
    chain down to ``depth`` is always kept; the remaining slots are filled with
    the best-scoring candidates whose parent is already in the tree (ties:
    shallower first, then lower parent, then lower rank).  Nodes are emitted in
    level order so that ``parent[i] < i``.
    """
    w = np.array([decay ** j for j in range(width)], dtype=np.float64)
    w /= w.sum()
    # node record: (path tuple of ranks)
    chosen = {(): 1.0}
    chain = ()
    for _ in range(depth):
        chain = chain + (0,)
        chosen[chain] = chosen[chain[:-1]] * w[0]
    if len(chosen) > n_nodes:
        raise ValueError("n_nodes smaller than the mandatory chain")
    heap: List = []
    counter = 0

    def push_children(path):
        nonlocal counter
        if len(path) >= depth:
            return
        for j in range(width):
            child = path + (j,)
            if child in chosen:
                continue
            score = chosen[path] * w[j]
            heapq.heappush(heap, (-score, len(child), path, j, counter))
            counter += 1

    for p in list(chosen):
        push_children(p)
    while len(chosen) < n_nodes and heap:
        negs, _, par, j, _ = heapq.heappop(heap)
        child = par + (j,)
        if child in chosen:
            continue
        chosen[child] = -negs
        push_children(child)
    order = sorted(chosen, key=lambda p: (len(p), p))
    index = {p: i for i, p in enumerate(order)}
    parent = [-1] + [index[p[:-1]] for p in order[1:]]
    rank = [0] + [p[-1] for p in order[1:]]
    return _finish_tree(parent, rank)


def random_tree(rng: np.random.Generator, n_nodes: int, max_depth: Optional[int] = None,
                max_children: Optional[int] = None) -> Dict[str, np.ndarray]:
    """``parent[i] ~ U[0, i)``, redrawn until the depth / fan-out limits hold."""
    for _ in range(100000):
        parent = [-1] + [int(rng.integers(0, i)) for i in range(1, n_nodes)]
        t = _finish_tree(parent, [0] * n_nodes)
        if max_depth is not None and int(t["depth"].max()) != max_depth:
            continue
        kids: Dict[int, int] = {}
        rank = [0] * n_nodes
        for i in range(1, n_nodes):
            rank[i] = kids.get(parent[i], 0)
            kids[parent[i]] = rank[i] + 1
        if max_children is not None and kids and max(kids.values()) > max_children:
            continue
        return _finish_tree(parent, rank)
    raise RuntimeError("could not draw a tree with the requested limits")


def chain_tree(n_nodes: int) -> Dict[str, np.ndarray]:
    return _finish_tree([-1] + list(range(n_nodes - 1)), [0] * n_nodes)


def star_tree(n_nodes: int) -> Dict[str, np.ndarray]:
    return _finish_tree([-1] + [0] * (n_nodes - 1), [0] + list(range(n_nodes - 1)))


# --------------------------------------------------------------------------
# Paged KV cache
# --------------------------------------------------------------------------
def make_kv_cache(rng: np.random.Generator, seq_lens: Sequence[int], n_nodes: Sequence[int],
                  n_visual: Sequence[int], n_kv_heads: int, head_dim: int = 128,
                  page_size: int = 64, n_layers: int = 1, shuffle: bool = False,
                  spare_frac: float = 0.0, visual_scale: float = 1.5,
                  poison: bool = True) -> Dict[str, np.ndarray]:
    """Paged bf16 K/V pools for a batch of sequences.

    Sequence b owns logical positions ``0 .. L_b + N_b - 1``: the prefix, whose
    first ``n_visual[b]`` rows are visual-token rows (N(0,1) * visual_scale) and
    the rest text rows (N(0,1)), followed by the K/V of this round's N_b tree
    nodes (N(0,1)).  Position t lives in page ``page_table[b, t // P]``, slot
    ``t % P``.  Pool layout: ``[layer, page, kv_head, slot, d]`` (uint16 bf16
    bits).  Rows that belong to no token hold a NaN pattern when ``poison``.
    """
    B = len(seq_lens)
    P = page_size
    tot = [int(seq_lens[b]) + int(n_nodes[b]) for b in range(B)]
    pages_b = [(t + P - 1) // P for t in tot]
    max_pages = max(pages_b)
    used = sum(pages_b)
    n_pages = int(np.ceil(used * (1.0 + spare_frac))) if spare_frac > 0 else used
    ids = rng.permutation(n_pages)[:used] if shuffle else np.arange(used)
    page_table = np.full((B, max_pages), -1, dtype=np.int32)
    c = 0
    for b in range(B):
        page_table[b, :pages_b[b]] = ids[c:c + pages_b[b]]
        c += pages_b[b]
    fill = POISON_BF16 if poison else np.uint16(0)
    shape = (n_layers, n_pages, n_kv_heads, P, head_dim)
    k_pool = np.full(shape, fill, dtype=np.uint16)
    v_pool = np.full(shape, fill, dtype=np.uint16)
    for layer in range(n_layers):
        for b in range(B):
            T = tot[b]
            for pool in (k_pool, v_pool):
                x = rng.standard_normal((T, n_kv_heads, head_dim), dtype=np.float32)
                x[:int(n_visual[b])] *= np.float32(visual_scale)
                bits = bf16_bits(x)
                for pg in range(pages_b[b]):
                    lo, hi = pg * P, min((pg + 1) * P, T)
                    # [tokens, heads, d] -> [heads, tokens, d]
                    pool[layer, page_table[b, pg], :, :hi - lo, :] = bits[lo:hi].transpose(1, 0, 2)
    return {"k_pool": k_pool, "v_pool": v_pool, "page_table": page_table,
            "seq_len": np.asarray(seq_lens, dtype=np.int32)}


def place_rows(pool: np.ndarray, page_table_row: np.ndarray, first_pos: int, rows: np.ndarray,
               page_size: int = 64) -> None:
    """Stores ``rows`` (uint16 [layers, tokens, kv_heads, d]) at logical positions ``first_pos ..`` of one
    sequence of a paged pool ``[layers, pages, kv_heads, slot, d]``, in place.  Stands in for the
    model forward that writes a round's tree K/V into the cache."""
    for i in range(rows.shape[1]):
        t = first_pos + i
        pool[:, int(page_table_row[t // page_size]), :, t % page_size, :] = rows[:, i]


def make_q(rng: np.random.Generator, sum_nodes: int, n_q_heads: int, head_dim: int = 128,
           n_layers: int = 1) -> np.ndarray:
    """Query rows ``[layer, node, q_head, d]`` ~ N(0,1), bf16 bits."""
    x = rng.standard_normal((n_layers, sum_nodes, n_q_heads, head_dim), dtype=np.float32)
    return bf16_bits(x)


# --------------------------------------------------------------------------
# Logits
# --------------------------------------------------------------------------
def make_logits(rng: np.random.Generator, rows: int, vocab: int, kind) -> Dict[str, np.ndarray]:
    """fp32 logits rows.

    ``kind`` is a string or a per-row list of strings:
      "low"   N(0,1) plus one planted peak = row max + U[6,10]   (low entropy)
      "high"  N(0,1) * 0.5, nothing planted                       (high entropy)
      "mixed" N(0,1) * s, s drawn from {0.5, 2, 8}, plus a planted peak
              = row max + U[0.5,4] at a random index
      "mid:<m>" N(0,1) plus a planted peak = row max + m           (tunable)
      "steps:<m>" N(0,1) plus eight planted peaks at row max + m, m - 1, m - 2, ...
              (a draft that has a clear first choice and plausible alternatives)
    """
    kinds = [kind] * rows if isinstance(kind, str) else list(kind)
    out = np.empty((rows, vocab), dtype=np.float32)
    peak = np.full(rows, -1, dtype=np.int32)
    for r in range(rows):
        kd = kinds[r]
        x = rng.standard_normal(vocab, dtype=np.float32)
        if kd == "high":
            x *= np.float32(0.5)
        elif kd == "mixed":
            x *= np.float32([0.5, 2.0, 8.0][int(rng.integers(0, 3))])
        if kd.startswith("steps:"):
            top = float(kd[6:])
            base = x.max()
            idx = rng.choice(vocab, size=8, replace=False)
            for j, ix in enumerate(idx):
                x[int(ix)] = np.float32(base + np.float32(top - j))
            peak[r] = int(idx[0])
        elif kd != "high":
            if kd == "low":
                margin = rng.uniform(6.0, 10.0)
            elif kd == "mixed":
                margin = rng.uniform(0.5, 4.0)
            elif kd.startswith("mid:"):
                margin = float(kd[4:])
            else:
                raise ValueError(kd)
            j = int(rng.integers(0, vocab))
            x[j] = np.float32(x.max() + np.float32(margin))
            peak[r] = j
        out[r] = x
    return {"logits": out, "peak": peak}


def make_target_logits(rng: np.random.Generator, tree: Dict[str, np.ndarray],
                       draft_token: np.ndarray, accept_node: int, vocab: int) -> Dict[str, np.ndarray]:
    """Target-model logits rows for one tree with a planted greedy path.

    Row p is N(0,1) with a peak (row max + U[6,10]) at a chosen token.  For every
    node p that is a proper ancestor of ``accept_node`` the peak sits on the
    draft token of p's child on that root path, so the greedy walk can follow
    the path down to ``accept_node``; every other row peaks at a random token.
    ``draft_token`` is an input (whoever calls this supplies it).
    """
    parent = tree["parent"]
    n = len(parent)
    want = rng.integers(0, vocab, size=n).astype(np.int64)
    c = int(accept_node)
    while parent[c] >= 0:
        want[parent[c]] = int(draft_token[c])
        c = int(parent[c])
    out = np.empty((n, vocab), dtype=np.float32)
    for r in range(n):
        x = rng.standard_normal(vocab, dtype=np.float32)
        x[want[r]] = np.float32(x.max() + np.float32(rng.uniform(6.0, 10.0)))
        out[r] = x
    return {"logits": out, "peak": want.astype(np.int32)}


def markov_entropy_states(rng: np.random.Generator, rounds: int, p_stay: float = 0.8) -> List[int]:
    """Two-state chain (0 = low entropy, 1 = high entropy) with P(stay) = p_stay."""
    s = int(rng.integers(0, 2))
    out = []
    for _ in range(rounds):
        out.append(s)
        if rng.random() >= p_stay:
            s = 1 - s
    return out


# --------------------------------------------------------------------------
# Synthetic acceptance process for multi-round decode loops.  The target model
# is replaced by a table of draws: for a node whose children sit at level l,
# the target's greedy token equals the draft's rank-R candidate with
# P(R = r) = p_l (1 - p_l)^r,  p_l = p * gamma^(l-1)   (r < k), and no candidate
# otherwise.  With a chain (only rank-0 children) level l is then accepted with
# probability p * gamma^(l-1), the process of the paper's expected-acceptance
# theorem (Section 4.2).  The table is data: both the CPU oracle loop and the
# device loop look the draws up, neither draws anything itself.
# --------------------------------------------------------------------------
NO_CANDIDATE = 255


def acceptance_picks(rng: np.random.Generator, rounds: int, n_slots: int, max_level: int, k: int,
                     p: float, gamma: float) -> np.ndarray:
    """uint8 [rounds, n_slots, max_level + 1]: entry [r, u, l] is the candidate rank the target agrees
    with at node slot u in round r if u's children are at level l (l >= 1; column 0 is unused), or
    NO_CANDIDATE."""
    out = np.full((rounds, n_slots, max_level + 1), NO_CANDIDATE, dtype=np.uint8)
    for lvl in range(1, max_level + 1):
        pl = float(p) * float(gamma) ** (lvl - 1)
        # number of failures before the first success of a Bernoulli(pl) sequence
        draws = rng.geometric(pl, size=(rounds, n_slots)) - 1 if pl > 0 else np.full((rounds, n_slots), k)
        out[:, :, lvl] = np.where(draws < k, draws, NO_CANDIDATE).astype(np.uint8)
    return out


def make_loop_logits(rng: np.random.Generator, rows: int, vocab: int, kind: str) -> np.ndarray:
    """Draft logits rows for the decode loops: as make_logits, with token 0 pushed far down so that it is
    never among a row's top candidates (the loops use it as the token that matches no draft node)."""
    lg = make_logits(rng, rows, vocab, kind)["logits"]
    lg[:, 0] = np.float32(-30.0)
    return lg


# --------------------------------------------------------------------------
# The five configurations
# --------------------------------------------------------------------------
def make_config(cfg: int, n_layers: Optional[int] = None, rounds: Optional[int] = None,
                scale_down: int = 1) -> Dict:
    """Inputs of configuration ``cfg`` (1..5).

    Returns a dict with the attention inputs (``q``, ``k_pool``, ``v_pool``,
    ``page_table``, ``seq_len``), the per-sequence trees (``trees``,
    ``node_offsets``) and the draft logits (``draft_logits`` with one row per
    node, ``k``, ``k_entropy``).  For configuration 4 the logits come as a list
    (one entry per round) with the Markov state of each round.  Target logits
    depend on the draft tokens and are built afterwards with
    :func:`make_target_logits`.

    ``scale_down`` divides the prefix lengths (tests use it to get a small case
    with the same structure); ``n_layers`` / ``rounds`` override the defaults.
    """
    if cfg == 1:
        Hq, Hkv, V, k, ke = 8, 1, 32000, 4, 4
        tree = random_tree(_rng(cfg, 0), 15, max_depth=4, max_children=4)
        trees, L, nvis = [tree], [256 // scale_down], [0]
        kv = make_kv_cache(_rng(cfg, 1), L, [15], nvis, Hkv, n_layers=n_layers or 1)
        logits = make_logits(_rng(cfg, 3), 15, V, "mixed")
        # one exact value tie inside the top-k of row 3 (lower index must win)
        lg = logits["logits"]
        a, b = sorted(int(v) for v in _rng(cfg, 4).choice(V, size=2, replace=False))
        if logits["peak"][3] in (a, b):
            a, b = a + 1, b + 1
        srt = np.sort(lg[3])
        tie = np.float32((srt[-1] + srt[-2]) * np.float32(0.5))
        lg[3, a] = tie
        lg[3, b] = tie
        draft = [logits]
        states = [0]
    elif cfg in (2, 3):
        Hq, Hkv, V = 64, 8, 152064
        if cfg == 2:
            tmpl, L0, nv0, kind, k, ke = TEMPLATES[0], 2048, 1600, "low", 2, 10
        else:
            tmpl, L0, nv0, kind, k, ke = TEMPLATES[3], 4096, 3200, "high", 10, 10
        tree = make_template(*tmpl)
        trees, L, nvis = [tree], [L0 // scale_down], [nv0 // scale_down]
        kv = make_kv_cache(_rng(cfg, 1), L, [tmpl[2]], nvis, Hkv, n_layers=n_layers or 1)
        draft = [make_logits(_rng(cfg, 3), tmpl[2], V, kind)]
        states = [0 if cfg == 2 else 1]
    elif cfg == 4:
        Hq, Hkv, V, k, ke = 64, 8, 152064, 10, 10
        N = 60
        L = [16384 // scale_down]
        nvis = [(32 * 196) // scale_down]
        # both templates of this configuration carry 60 nodes
        trees = [make_template(8, 2, N)]
        kv = make_kv_cache(_rng(cfg, 1), L, [N], nvis, Hkv, n_layers=n_layers or 3,
                           shuffle=True, spare_frac=0.125)
        # the first seeded chain (tensor ids 5, 6, ...) that visits both states
        for tid in range(5, 30):
            states = markov_entropy_states(_rng(cfg, 50 + tid), rounds or 8, 0.8)
            if len(set(states)) == 2 or (rounds or 8) < 2:
                break
        draft = [make_logits(_rng(cfg, 100 + r), N, V, "low" if s == 0 else "high")
                 for r, s in enumerate(states)]
    elif cfg == 5:
        Hq, Hkv, V, k, ke = 64, 8, 152064, 10, 10
        B = 16
        r = _rng(cfg, 0)
        L = [int(v) // scale_down for v in r.integers(1024, 8193, size=B)]
        nvis = [int(0.6 * l) for l in L]
        # entropy band per sequence, cycling through all four templates
        band = [int(v) for v in r.permutation(B) % 4]
        trees = [make_template(*TEMPLATES[t]) for t in band]
        kv = make_kv_cache(_rng(cfg, 1), L, [len(t["parent"]) for t in trees], nvis, Hkv,
                           n_layers=n_layers or 1, shuffle=True, spare_frac=0.1)
        # planted margins that land alpha in the four bands (>=0.8, 0.4-0.8, 0.1-0.4, <0.1)
        kinds_by_band = ["low", "mid:3.0", "mid:1.8", "high"]
        rows = []
        for b in range(B):
            rows.extend([kinds_by_band[band[b]]] * len(trees[b]["parent"]))
        draft = [make_logits(_rng(cfg, 3), len(rows), V, rows)]
        states = band
    else:
        raise ValueError("config must be 1..5")
    n_nodes = [len(t["parent"]) for t in trees]
    node_offsets = np.concatenate([[0], np.cumsum(n_nodes)]).astype(np.int32)
    nl = kv["k_pool"].shape[0]
    q = make_q(_rng(cfg, 2), int(node_offsets[-1]), Hq, 128, nl)
    root_token = _rng(cfg, 6).integers(0, V, size=len(trees)).astype(np.int32)
    return {
        "cfg": cfg, "name": CONFIG_NAMES[cfg],
        "n_q_heads": Hq, "n_kv_heads": Hkv, "head_dim": 128, "page_size": 64, "vocab": V,
        "k": k, "k_entropy": ke, "sm_scale": float(1.0 / np.sqrt(128.0)),
        "trees": trees, "node_offsets": node_offsets, "root_token": root_token,
        "parent": np.concatenate([t["parent"] for t in trees]).astype(np.int32),
        "rank": np.concatenate([t["rank"] for t in trees]).astype(np.int32),
        "q": q, **kv,
        "draft_logits": [d["logits"] for d in draft], "draft_peak": [d["peak"] for d in draft],
        "states": states,
    }
