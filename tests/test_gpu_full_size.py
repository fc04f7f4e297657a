"""GPU parity at the benchmark's full size and launch configuration: 80 stacked layers,
16384-token prefix with a shuffled page table, 60-node tree, 64/8/128 heads.

The fp64 oracle cannot redo 80 layers in test time, so three sampled layers are compared
with it element by element (on the very bytes the GPU used), and properties that hold at
any size cover the rest: every output finite, every layer of the compacted cache equal to
the input except for the accepted rows, which must be copies of their source rows.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_00523_b200 as sage
from helpers import check_attention, dev_i32, host_bits
from workloads import make_template
from workloads.gen import _rng

pytestmark = pytest.mark.gpu

HQ, HKV, D, P = 64, 8, 128, 64
N_LAYERS, L, N, N_VISUAL = 80, 16384, 60, 32 * 196
SAMPLED_LAYERS = (0, 37, 79)


def _build(n_nodes=N, shape=(3, 10)):
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev)
    gen.manual_seed(523000 + 4000 + 77)
    used = (L + n_nodes + P - 1) // P
    n_pages = int(np.ceil(used * 1.125))
    perm = _rng(4, 1).permutation(n_pages)[:used].astype(np.int32)
    k = torch.empty((N_LAYERS, n_pages, HKV, P, D), dtype=torch.bfloat16, device=dev)
    v = torch.empty_like(k)
    vis = torch.from_numpy(perm[:N_VISUAL // P].astype(np.int64)).to(dev)
    for pool in (k, v):
        for layer in range(N_LAYERS):
            pool[layer].normal_(generator=gen)
            pool[layer, vis] *= 1.5
    q = torch.empty((N_LAYERS, n_nodes, HQ, D), dtype=torch.bfloat16, device=dev).normal_(generator=gen)
    tree = make_template(shape[0], shape[1], n_nodes)
    return dict(k=k, v=v, q=q, perm=perm, tree=tree, page_table=dev_i32(perm.reshape(1, -1)),
                seq_len=dev_i32([L]), parent=dev_i32(tree["parent"]), offs=dev_i32([0, n_nodes]))


@pytest.mark.parametrize("schedule", [0, 1, 3], ids=["as_benchmarked", "streaming", "pairs"])
def test_attention_80_layers_sampled_layers_match_the_oracle_and_all_outputs_are_finite(schedule):
    w = _build()
    sage.sage_debug_attention_schedule(schedule)
    st = sage.new_status()
    out = sage.sage_tree_attention(w["q"], w["k"], w["v"], w["page_table"], w["seq_len"], w["parent"], w["offs"],
                                   1.0 / np.sqrt(D), status=st)
    torch.cuda.synchronize()
    sage.sage_debug_attention_schedule(0)
    assert int(st.item()) == 0, sage.status_string(int(st.item()))
    assert bool(torch.isfinite(out.float()).all())
    offs = np.array([0, N], np.int32)
    for layer in SAMPLED_LAYERS:
        want = oracle.tree_attention(host_bits(w["q"][layer]), host_bits(w["k"][layer]), host_bits(w["v"][layer]),
                                     w["perm"].reshape(1, -1), np.array([L], np.int32), w["tree"]["parent"], offs,
                                     HQ, HKV, D, P, 1.0 / np.sqrt(D))
        check_attention(host_bits(out[layer]), want)


@pytest.mark.parametrize("n_nodes,shape", [(16, (8, 2)), (24, (8, 2))], ids=["16_nodes", "24_nodes"])
def test_attention_80_layers_deep_narrow_trees(n_nodes, shape):
    """The HBM-bound regime of the benchmark: deep, narrow trees of one (16 nodes) and two (24 nodes) row tiles,
    in the launch configuration the library picks for them."""
    w = _build(n_nodes, shape)
    st = sage.new_status()
    out = sage.sage_tree_attention(w["q"], w["k"], w["v"], w["page_table"], w["seq_len"], w["parent"], w["offs"],
                                   1.0 / np.sqrt(D), status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0, sage.status_string(int(st.item()))
    assert bool(torch.isfinite(out.float()).all())
    offs = np.array([0, n_nodes], np.int32)
    for layer in SAMPLED_LAYERS:
        want = oracle.tree_attention(host_bits(w["q"][layer]), host_bits(w["k"][layer]), host_bits(w["v"][layer]),
                                     w["perm"].reshape(1, -1), np.array([L], np.int32), w["tree"]["parent"], offs,
                                     HQ, HKV, D, P, 1.0 / np.sqrt(D))
        check_attention(host_bits(out[layer]), want)


@pytest.mark.parametrize("n_nodes,shape", [(9, (8, 1)), (24, (8, 2)), (60, (3, 10))], ids=["9_nodes", "24_nodes", "60_nodes"])
def test_attention_80_layers_node_arrays_of_full_capacity(n_nodes, shape):
    """A decode loop that lives on the device keeps node arrays of full capacity (64 nodes) whatever the
    tree of a round looks like, so the host only knows an upper bound of the tree size: the library then
    starts every kernel that might apply and the tree size found on the device (node_offsets) picks the one
    that runs.  The rows past the tree must stay untouched."""
    cap = sage.SAGE_MAX_NODES
    w = _build(n_nodes, shape)
    dev = w["q"].device
    q = torch.zeros((N_LAYERS, cap, HQ, D), dtype=torch.bfloat16, device=dev)
    q[:, :n_nodes] = w["q"]
    parent = np.full(cap, -1, np.int32)
    parent[:n_nodes] = w["tree"]["parent"]
    out = torch.full_like(q, 7.0)
    st = sage.new_status()
    sage.sage_tree_attention(q, w["k"], w["v"], w["page_table"], w["seq_len"], dev_i32(parent), w["offs"],
                             1.0 / np.sqrt(D), out=out, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0, sage.status_string(int(st.item()))
    assert bool((out[:, n_nodes:].float() == 7.0).all())
    assert bool(torch.isfinite(out[:, :n_nodes].float()).all())
    offs = np.array([0, n_nodes], np.int32)
    for layer in (SAMPLED_LAYERS[0], SAMPLED_LAYERS[-1]):
        want = oracle.tree_attention(host_bits(q[layer, :n_nodes]), host_bits(w["k"][layer]), host_bits(w["v"][layer]),
                                     w["perm"].reshape(1, -1), np.array([L], np.int32), w["tree"]["parent"], offs,
                                     HQ, HKV, D, P, 1.0 / np.sqrt(D))
        check_attention(host_bits(out[layer, :n_nodes]), want)


def test_compaction_80_layers_moves_exactly_the_accepted_rows():
    w = _build()
    k0, v0 = w["k"].clone(), w["v"].clone()
    # a root path of the tree: from the root, always to the last child (far from its destination slot)
    parent = w["tree"]["parent"]
    path = [0]
    while len(path) < 4:
        kids = [i for i in range(N) if parent[i] == path[-1]]
        if not kids:
            break
        path.append(kids[-1])
    max_path = 9
    path_arr = np.full((1, max_path), -1, np.int32)
    path_arr[0, :len(path)] = path
    st = sage.new_status()
    seq = w["seq_len"].clone()
    sage.sage_compact_kv(w["k"], w["v"], w["page_table"], seq, dev_i32(path_arr), dev_i32([len(path)]), status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and int(seq.item()) == L + len(path)
    # sampled layers against the oracle, byte for byte
    for layer in SAMPLED_LAYERS:
        wk, wv, wl = oracle.compact_kv(host_bits(k0[layer:layer + 1]), host_bits(v0[layer:layer + 1]),
                                       w["perm"].reshape(1, -1), np.array([L], np.int32), path_arr,
                                       np.array([len(path)], np.int32), P)
        assert np.array_equal(host_bits(w["k"][layer:layer + 1]), wk)
        assert np.array_equal(host_bits(w["v"][layer:layer + 1]), wv)
        assert int(wl[0]) == L + len(path)
    # every layer: destination rows are copies of their sources, nothing else changed
    for new, old in ((w["k"], k0), (w["v"], v0)):
        expect = old.clone()
        for j, node in enumerate(path):
            src, dst = L + node, L + j
            expect[:, int(w["perm"][dst // P]), :, dst % P, :] = old[:, int(w["perm"][src // P]), :, src % P, :]
        assert torch.equal(new.view(torch.int16), expect.view(torch.int16))
