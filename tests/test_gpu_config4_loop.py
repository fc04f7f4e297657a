"""Configuration 4 as a loop: eight decode rounds chained the way Algorithm 1 orders them, the
CUDA library against the fp64 oracle at every step of every round.

Round r (Section 3.3, phases 1-3; Section 3.2 "Temporal Correlation Exploitation"):
  draft logits of round r  -> sage_expand_topk   top-10 ids, alpha, draft tokens of the CURRENT tree
  alpha                    -> sage_select_tree   template of the NEXT round, handed over on the device
  q, paged K/V (16384+)    -> sage_tree_attention with the tree handed over by round r-1
                              (round 0: alpha = 0.5 -> template 0), two layers, full context
  target logits            -> sage_expand_topk(k=1)   the target's greedy token per node
  -> sage_accept -> sage_compact_kv; the bonus token becomes the next round's root token.
The device state (pools, seq_len, tree buffers, root token) is carried from round to round without
being refreshed from the host; only the round's new inputs (logits, q, the tree's K/V rows) are
uploaded, as a model forward would produce them.  The oracle runs the same loop on the CPU and
every round's top-k ids, template id, handed-over parent / rank arrays, attention outputs, path,
tau + 1, bonus token, sequence length and the whole compacted pools must agree.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_00523_b200 as sage
from helpers import (ENTROPY_ABS, check_attention, check_logits, dev_bf16, dev_f32, dev_i32, host_bits)
from workloads import bf16_bits, make_kv_cache, make_logits, make_q, make_target_logits, make_template, \
    markov_entropy_states, place_rows
from workloads.gen import POISON_BF16, _rng

pytestmark = pytest.mark.gpu

CFG = 4
HQ, HKV, D, P, V = 64, 8, 128, 64, 152064
N, L0, LAYERS, ROUNDS, MAX_PATH, K, KE = 60, 16384, 2, 8, 9, 10, 10
THR = [0.5]
SHAPES = [(8, 2, N), (3, 10, N)]          # template 0: deep-narrow (alpha >= 0.5); template 1: shallow-wide


def test_config4_eight_round_lookahead_loop_matches_the_oracle():
    tmpl = [make_template(*s) for s in SHAPES]
    for tid in range(5, 30):                                   # the configuration's seeded chain
        states = markov_entropy_states(_rng(CFG, 50 + tid), ROUNDS, 0.8)
        if len(set(states)) == 2:
            break
    # cache: 16384-token prefix on shuffled pages, with room for eight rounds of accepted tokens
    kv = make_kv_cache(_rng(CFG, 1), [L0], [N + ROUNDS * MAX_PATH], [32 * 196], HKV, n_layers=LAYERS, shuffle=True,
                       spare_frac=0.125)
    pt = kv["page_table"]
    k_h, v_h = kv["k_pool"], kv["v_pool"]
    poison = np.full((LAYERS, N + ROUNDS * MAX_PATH, HKV, D), POISON_BF16, np.uint16)
    place_rows(k_h, pt[0], L0, poison)                          # nothing beyond the prefix is valid yet
    place_rows(v_h, pt[0], L0, poison)
    seq_h = np.array([L0], np.int32)
    offs = np.array([0, N], np.int32)

    k_d, v_d = dev_bf16(k_h), dev_bf16(v_h)
    pt_d, seq_d, offs_d = dev_i32(pt), dev_i32(seq_h), dev_i32(offs)
    alpha_row = dev_i32([0])
    bank_p = np.full((2, 64), -1, np.int32)
    bank_r = np.zeros((2, 64), np.int32)
    for i, t in enumerate(tmpl):
        bank_p[i, :N], bank_r[i, :N] = t["parent"], t["rank"]
    bank_p_d, bank_r_d, bank_n_d = dev_i32(bank_p), dev_i32(bank_r), dev_i32([N, N])
    policy = sage.make_policy(THR)
    status = sage.new_status()

    # round 0 starts from alpha = 0.5 (Algorithm 1's initial confidence)
    tid_h = int(oracle.select_tree(np.float32([0.5]), THR)[0][0])
    assert tid_h == 0
    cur = {"next_parent": dev_i32(bank_p[tid_h]), "next_rank": dev_i32(bank_r[tid_h])}
    root_h = _rng(CFG, 6).integers(0, V, size=1).astype(np.int32)
    root_d = dev_i32(root_h)
    seen_templates = []

    for r in range(ROUNDS):
        tree = tmpl[tid_h]
        L = int(seq_h[0])
        # ---- this round's inputs, as the model forwards would deliver them
        lg = make_logits(_rng(CFG, 100 + r), N, V, "low" if states[r] == 0 else "high")["logits"]
        q_bits = make_q(_rng(CFG, 400 + r), N, HQ, D, LAYERS)
        rk = _rng(CFG, 300 + r)
        tree_k = bf16_bits(rk.standard_normal((LAYERS, N, HKV, D), dtype=np.float32))
        tree_v = bf16_bits(rk.standard_normal((LAYERS, N, HKV, D), dtype=np.float32))
        place_rows(k_h, pt[0], L, tree_k)
        place_rows(v_h, pt[0], L, tree_v)
        assert int(seq_d.item()) == L
        tk_d, tv_d = dev_bf16(tree_k), dev_bf16(tree_v)
        for i in range(N):                                      # same placement on the device-resident pools
            pg, slot = int(pt[0, (L + i) // P]), (L + i) % P
            k_d[:, pg, :, slot, :] = tk_d[:, i]
            v_d[:, pg, :, slot, :] = tv_d[:, i]

        # ---- phase 1 / 3: top-k expansion of the current tree and the confidence of this round
        got = sage.sage_expand_topk(dev_f32(lg), K, KE, parent=cur["next_parent"][:N], rank=cur["next_rank"][:N],
                                    node_offsets=offs_d, root_token=root_d, status=status)
        got = {n: t.cpu().numpy() for n, t in got.items()}
        check_logits(got, lg, K, KE)
        want_idx = oracle.topk(lg, K)
        want_tok = oracle.expand_gather(want_idx, tree["parent"], tree["rank"], offs, root_h)
        np.testing.assert_array_equal(got["draft_token"], want_tok)
        _, alpha_h = oracle.confidence(lg, KE)
        assert abs(float(got["alpha"][0]) - float(alpha_h[0])) <= ENTROPY_ABS
        assert abs(float(alpha_h[0]) - THR[0]) > 1e-4            # far from the threshold on both sides
        nxt = sage.sage_select_tree(dev_f32(got["alpha"]), policy, alpha_row=alpha_row, bank_parent=bank_p_d,
                                    bank_rank=bank_r_d, bank_n_nodes=bank_n_d, handover=True, status=status)
        next_tid_h = int(oracle.select_tree(alpha_h[:1].astype(np.float32), THR)[0][0])
        assert int(nxt["template_id"].item()) == next_tid_h
        assert next_tid_h == (0 if states[r] == 0 else 1)
        np.testing.assert_array_equal(nxt["next_parent"].cpu().numpy()[:N], tmpl[next_tid_h]["parent"])
        np.testing.assert_array_equal(nxt["next_rank"].cpu().numpy()[:N], tmpl[next_tid_h]["rank"])
        np.testing.assert_array_equal(nxt["next_node_offsets"].cpu().numpy(), offs)

        # ---- phase 2: verification attention with the tree handed over by the previous round
        out = sage.sage_tree_attention(dev_bf16(q_bits), k_d, v_d, pt_d, seq_d, cur["next_parent"][:N], offs_d,
                                       1.0 / np.sqrt(D), status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, sage.status_string(int(status.item()))
        out_bits = host_bits(out)
        for layer in range(LAYERS):
            want = oracle.tree_attention(q_bits[layer], k_h[layer], v_h[layer], pt, seq_h, tree["parent"], offs,
                                         HQ, HKV, D, P, 1.0 / np.sqrt(D))
            check_attention(out_bits[layer], want)

        # ---- target argmax, acceptance, cache update
        rr = _rng(CFG, 200 + r)
        leaf = int(rr.integers(1, N))
        tl = make_target_logits(rr, tree, want_tok, leaf, V)["logits"]
        tgt = sage.sage_expand_topk(dev_f32(tl), 1, 1, status=status)["topk_idx"]
        want_tgt = oracle.topk(tl, 1)[:, 0]
        np.testing.assert_array_equal(tgt.cpu().numpy()[:, 0], want_tgt)
        acc = sage.sage_accept(cur["next_parent"][:N], dev_i32(got["draft_token"]), tgt.reshape(-1).contiguous(),
                               offs_d, MAX_PATH, status=status)
        w_path, w_len, w_bonus = oracle.accept(tree["parent"], want_tok, want_tgt, offs, MAX_PATH)
        np.testing.assert_array_equal(acc["path"].cpu().numpy(), w_path)
        np.testing.assert_array_equal(acc["path_len"].cpu().numpy(), w_len)
        np.testing.assert_array_equal(acc["bonus_token"].cpu().numpy(), w_bonus)
        assert int(w_len[0]) > 1                                 # the planted path was followed
        sage.sage_compact_kv(k_d, v_d, pt_d, seq_d, acc["path"], acc["path_len"], status=status)
        k_h, v_h, seq_h = oracle.compact_kv(k_h, v_h, pt, seq_h, w_path, w_len, P)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        np.testing.assert_array_equal(seq_d.cpu().numpy(), seq_h)
        assert np.array_equal(host_bits(k_d), k_h)
        assert np.array_equal(host_bits(v_d), v_h)

        # ---- look-ahead: the tree chosen now is the next round's tree; the bonus token its root
        seen_templates.append(tid_h)
        cur, tid_h = nxt, next_tid_h
        root_d, root_h = acc["bonus_token"], w_bonus.astype(np.int32)
    assert len(set(seen_templates)) == 2                         # the loop really switched templates
    assert int(seq_h[0]) > L0 + ROUNDS
