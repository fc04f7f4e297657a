"""Multi-round decode loop on the device: Algorithm 1 of the paper with the two models replaced by
synthetic stand-ins, every step of the method running in the library's kernels and no host round
trip between rounds.

Round r (Section 3.3):
  phase 1  draft distribution of every node slot -> sage_expand_topk (top-k candidates, confidence alpha)
           tree of this round: a fixed tree (chain or static template), a template chosen by the
           previous round's alpha (sage_select_tree hand-over), or a tree grown level by level from the
           candidates (sage_grow_tree; depth / width from the previous round's alpha, maximum depth
           from the acceptance history)
  phase 2  sage_tree_attention over the paged cache; the target's greedy token per node
           (sage_expand_topk, k = 1, on the target logits); sage_accept; sage_compact_kv
  phase 3  alpha of this round is kept for the next tree (look-ahead, Section 3.2);
           sage_update_history turns tau into the next maximum depth (Section 3.3)

The models' stand-ins are data: the draft logits of each round are given, and the target's logits are
a fixed noise matrix with one planted peak per row, placed by `SyntheticTarget` from a table of
pre-drawn agreement ranks (workloads.acceptance_picks).  Placing that peak is the only arithmetic
here that is not a library call; it takes the place of the target model, not of a step of the method.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as sage

CAP = sage.SAGE_MAX_NODES
NO_CANDIDATE = 255
MISS_TOKEN = 0          # never among the draft candidates (workloads.make_loop_logits keeps it out)


class SyntheticTarget:
    """Target logits [CAP, V] whose greedy token at node u is the draft token of u's child of rank
    picks[r, u, depth(u) + 1] when the tree has such a child, and MISS_TOKEN otherwise."""

    def __init__(self, noise: torch.Tensor, picks: np.ndarray, k: int):
        self.logits = noise                                  # fp32 [CAP, V], values well below the planted peak
        self.picks = torch.from_numpy(picks.astype(np.int64)).to(noise.device)    # [R, CAP, levels + 1]
        self.k = k
        self.rows = torch.arange(CAP, device=noise.device)
        self.saved = torch.empty(CAP, dtype=torch.float32, device=noise.device)
        self.want = torch.zeros(CAP, dtype=torch.int64, device=noise.device)

    def plant(self, r: int, parent: torch.Tensor, rank: torch.Tensor, depth: torch.Tensor, n_nodes: torch.Tensor,
              draft_token: torch.Tensor) -> torch.Tensor:
        """All arguments are device tensors of capacity CAP (n_nodes: [1]); no host synchronisation."""
        k, rows = self.k, self.rows
        valid = (rows < n_nodes) & (rows > 0)
        # child_of[u * k + rank] = index of u's child with that rank, -1 if there is none
        flat = torch.where(valid, parent.long().clamp(min=0) * k + rank.long(), torch.full_like(rows, CAP * k))
        child_of = torch.full((CAP * k + 1,), -1, dtype=torch.int64, device=rows.device)
        child_of[flat] = torch.where(valid, rows, torch.full_like(rows, -1))
        child_of[CAP * k] = -1
        levels = self.picks.shape[2] - 1
        pick = self.picks[r % self.picks.shape[0]][rows, (depth.long() + 1).clamp(max=levels)]
        child = torch.where(pick < k, child_of[rows * k + pick.clamp(max=k - 1)], torch.full_like(rows, -1))
        child = torch.where(rows < n_nodes, child, torch.full_like(rows, -1))
        self.want = torch.where(child >= 0, draft_token.long()[child.clamp(min=0)], torch.full_like(rows, MISS_TOKEN))
        self.saved.copy_(self.logits[rows, self.want])
        self.logits[rows, self.want] = 50.0
        return self.logits

    def restore(self):
        self.logits[self.rows, self.want] = self.saved


class DecodeLoop:
    """One sequence, `policy` in {"chain", "static", "templates", "dynamic"}."""

    def __init__(self, *, policy: str, draft_logits: List[torch.Tensor], target: SyntheticTarget, k: int, k_entropy: int,
                 q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: torch.Tensor, prefix_len: int,
                 max_path: int, trees: Optional[List[Dict[str, np.ndarray]]] = None, thresholds=(), n_budget: int = CAP,
                 levels: int = 8, tree_policy_kw: Optional[dict] = None, history_kw: Optional[dict] = None,
                 root_token: int = 1, rounds_capacity: int = 4096):
        dev = q.device
        self.dev, self.policy, self.k, self.ke, self.max_path = dev, policy, k, k_entropy, max_path
        self.draft_logits, self.target = draft_logits, target
        self.q, self.k_pool, self.v_pool, self.page_table = q, k_pool, v_pool, page_table
        self.seq_len = torch.tensor([prefix_len], dtype=torch.int32, device=dev)
        self.n_budget, self.levels = n_budget, levels
        self.status = sage.new_status(dev)
        self.root_token = torch.tensor([root_token], dtype=torch.int32, device=dev)
        self.alpha_prev = torch.tensor([0.5], dtype=torch.float32, device=dev)       # Algorithm 1's initial confidence
        self.node_offsets = torch.zeros(2, dtype=torch.int32, device=dev)
        self.n_nodes = torch.ones(1, dtype=torch.int32, device=dev)
        self.tree_policy = sage.make_policy(list(thresholds), **(tree_policy_kw or {}))
        hk = dict(window=10, lower=2.0, upper=3.0, step=1.0, d_lo=3.0, d_hi=8.0)
        hk.update(history_kw or {})
        self.hist_policy = sage.make_history_policy(**hk)
        self.window_buf = torch.zeros((1, hk["window"]), dtype=torch.int32, device=dev)
        self.hist_count = torch.zeros(1, dtype=torch.int32, device=dev)
        self.d_max = torch.tensor([float((tree_policy_kw or {}).get("d_max", 8.0))], dtype=torch.float32, device=dev)
        self.alpha_row = torch.zeros(1, dtype=torch.int32, device=dev)
        rows, V = draft_logits[0].shape
        assert rows == CAP
        self.ws_topk = torch.empty(sage.sage_expand_topk_workspace_size(CAP, V), dtype=torch.uint8, device=dev)
        n_layers, _, Hq, d = q.shape
        self.ws_attn = torch.empty(sage.sage_tree_attention_workspace_size(n_layers, 1, CAP, Hq, k_pool.shape[2], d,
                                                                            page_table.shape[1]), dtype=torch.uint8, device=dev)
        self.attn_out = torch.empty_like(q)
        self.out_draft, self.out_target, self.out_accept, self.out_select = {}, {}, {}, {}
        self.tree = {"parent": torch.full((CAP,), -1, dtype=torch.int32, device=dev),
                     "rank": torch.zeros(CAP, dtype=torch.int32, device=dev),
                     "depth": torch.zeros(CAP, dtype=torch.int32, device=dev),
                     "token": torch.zeros(CAP, dtype=torch.int32, device=dev),
                     "cum_logprob": torch.zeros(CAP, dtype=torch.float32, device=dev),
                     "n_nodes": self.n_nodes, "frontier_begin": torch.zeros(1, dtype=torch.int32, device=dev)}
        if policy in ("chain", "static", "templates"):
            assert trees
            nt = len(trees)
            bank_p = np.full((nt, CAP), -1, np.int32)
            bank_r = np.zeros((nt, CAP), np.int32)
            bank_d = np.zeros((nt, CAP), np.int32)
            bank_n = np.zeros(nt, np.int32)
            for i, t in enumerate(trees):
                n = len(t["parent"])
                bank_p[i, :n], bank_r[i, :n], bank_d[i, :n], bank_n[i] = t["parent"], t["rank"], t["depth"], n
            self.bank_parent, self.bank_rank = torch.from_numpy(bank_p).to(dev), torch.from_numpy(bank_r).to(dev)
            self.bank_depth, self.bank_n = torch.from_numpy(bank_d).to(dev), torch.from_numpy(bank_n).to(dev)
            self.template_id = torch.zeros(1, dtype=torch.int32, device=dev)
            self._load_template_tree()
        # per-round records, written on the device
        self.rec = {"path_len": torch.zeros(rounds_capacity, dtype=torch.int32, device=dev),
                    "n_nodes": torch.zeros(rounds_capacity, dtype=torch.int32, device=dev),
                    "bonus": torch.zeros(rounds_capacity, dtype=torch.int32, device=dev),
                    "d_max": torch.zeros(rounds_capacity, dtype=torch.float32, device=dev),
                    "alpha": torch.zeros(rounds_capacity, dtype=torch.float32, device=dev),
                    "template": torch.zeros(rounds_capacity, dtype=torch.int32, device=dev),
                    "seq_len": torch.zeros(rounds_capacity, dtype=torch.int32, device=dev),
                    "path": torch.zeros((rounds_capacity, max_path), dtype=torch.int32, device=dev),
                    "tree_parent": torch.zeros((rounds_capacity, CAP), dtype=torch.int32, device=dev),
                    "draft_token": torch.zeros((rounds_capacity, CAP), dtype=torch.int32, device=dev)}
        self.round = 0

    def _load_template_tree(self):
        """The tree of the current template id (a device tensor) becomes the tree of the round."""
        tid = self.template_id.long()
        self.tree["parent"].copy_(self.bank_parent.index_select(0, tid)[0])
        self.tree["rank"].copy_(self.bank_rank.index_select(0, tid)[0])
        self.tree["depth"].copy_(self.bank_depth.index_select(0, tid)[0])
        self.n_nodes.copy_(self.bank_n.index_select(0, tid))

    def step(self):
        r, st, tree = self.round, self.status, self.tree
        draft = self.draft_logits[r % len(self.draft_logits)]
        if self.policy == "dynamic":
            d = sage.sage_expand_topk(draft, self.k, self.ke, out=self.out_draft, ws=self.ws_topk, status=st)
            # a fresh tree: the root is the last committed token
            tree["parent"].fill_(-1); tree["rank"].zero_(); tree["depth"].zero_(); tree["cum_logprob"].zero_()
            tree["token"][:1].copy_(self.root_token)
            self.n_nodes.fill_(1); tree["frontier_begin"].zero_()
            for _ in range(self.levels):
                sage.sage_grow_tree(d["topk_idx"], d["topk_logprob"], self.alpha_prev, self.tree_policy, tree,
                                    n_max=self.n_budget, d_max_seq=self.d_max, status=st)
            self.node_offsets[1:].copy_(self.n_nodes)
            draft_token = tree["token"]
        else:
            self.node_offsets[1:].copy_(self.n_nodes)
            d = sage.sage_expand_topk(draft, self.k, self.ke, parent=tree["parent"], rank=tree["rank"],
                                      node_offsets=self.node_offsets, root_token=self.root_token, out=self.out_draft,
                                      ws=self.ws_topk, status=st)
            draft_token = d["draft_token"]
        # ---- phase 2: verification
        tl = self.target.plant(r, tree["parent"], tree["rank"], tree["depth"], self.n_nodes, draft_token)
        sage.sage_tree_attention(self.q, self.k_pool, self.v_pool, self.page_table, self.seq_len, tree["parent"],
                                 self.node_offsets, 1.0 / np.sqrt(self.q.shape[3]), out=self.attn_out, ws=self.ws_attn, status=st)
        t = sage.sage_expand_topk(tl, 1, 1, out=self.out_target, ws=self.ws_topk, status=st)
        a = sage.sage_accept(tree["parent"], draft_token, t["topk_idx"], self.node_offsets, self.max_path,
                             out=self.out_accept, status=st)
        self.target.restore()
        sage.sage_compact_kv(self.k_pool, self.v_pool, self.page_table, self.seq_len, a["path"], a["path_len"], status=st)
        # ---- records of the round (device-side copies)
        rec = self.rec
        rec["path_len"][r:r + 1].copy_(a["path_len"]); rec["bonus"][r:r + 1].copy_(a["bonus_token"])
        rec["n_nodes"][r:r + 1].copy_(self.n_nodes); rec["alpha"][r:r + 1].copy_(d["alpha"][:1])
        rec["seq_len"][r:r + 1].copy_(self.seq_len); rec["path"][r].copy_(a["path"][0])
        rec["tree_parent"][r].copy_(tree["parent"]); rec["draft_token"][r].copy_(draft_token)
        # ---- phase 3: the next round's tree parameters
        sage.sage_update_history(a["path_len"], self.hist_policy, self.window_buf, self.hist_count, self.d_max, status=st)
        rec["d_max"][r:r + 1].copy_(self.d_max)
        if self.policy == "templates":
            # the template for the next round and its parent / rank arrays, handed over by the library
            o = sage.sage_select_tree(d["alpha"], self.tree_policy, alpha_row=self.alpha_row, bank_parent=self.bank_parent,
                                      bank_rank=self.bank_rank, bank_n_nodes=self.bank_n, handover=True, out=self.out_select,
                                      status=st)
            self.template_id.copy_(o["template_id"])
            rec["template"][r:r + 1].copy_(self.template_id)
            tree["parent"].copy_(o["next_parent"][:CAP]); tree["rank"].copy_(o["next_rank"][:CAP])
            self.n_nodes.copy_(o["next_node_offsets"][1:2])
            tree["depth"].copy_(self.bank_depth.index_select(0, self.template_id.long())[0])   # for the stand-in target only
        self.alpha_prev.copy_(d["alpha"][:1])
        self.root_token.copy_(a["bonus_token"])
        self.round += 1

    def run(self, rounds: int):
        for _ in range(rounds):
            self.step()
        return self.rec
