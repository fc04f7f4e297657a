"""sage_expand_topk_static: the entry point for callers that cannot allocate.

Some users of this library run where device allocation is off the table: a plug-in
inside a serving engine whose memory pool has already claimed the whole GPU gets its
input and output buffers and nothing else, and a decode loop cannot afford cudaMalloc's
device-wide synchronisation.  For them the library carries its own fixed scratch array.
These tests call that entry point through the C ABI, twice in a row on different inputs
(the array is shared between calls and keeps the previous call's contents), and compare
every output with what the caller-workspace entry point gives on the same inputs and with
the CPU oracle.

The file name sorts after every other test file on purpose: a run that stops at the
first failure has then already gone through all the other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2602_00523_b200 as sage
from helpers import ENTROPY_ABS, check_logits, dev_f32, dev_i32
from workloads import make_logits, make_template

FLOAT_OUTPUTS = ("topk_logprob", "entropy_full", "entropy_topk", "alpha", "lse")


def _outputs(rows, k, n_nodes, dev):
    o = {"topk_idx": torch.full((rows, k), -7, dtype=torch.int32, device=dev),
         "topk_logprob": torch.full((rows, k), float("nan"), dtype=torch.float32, device=dev),
         "draft_token": torch.full((n_nodes,), -7, dtype=torch.int32, device=dev)}
    for name in ("entropy_full", "entropy_topk", "alpha", "lse"):
        o[name] = torch.full((rows,), float("nan"), dtype=torch.float32, device=dev)
    return o


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_on_two_calls_in_a_row():
    dev = torch.device("cuda")
    rng = np.random.Generator(np.random.Philox(52399))
    # call 1: 60 high-entropy rows of the full vocabulary, k = 10, with the expansion gather;
    # call 2: 24 low-entropy rows of a ragged vocabulary, k = 2.  The second call uses fewer
    # and differently sized scratch slots than the first, so stale contents would show.
    cases = [(make_template(3, 10, 60), 152064, "high", 10, 10),
             (make_template(8, 2, 24), 40961, "low", 2, 10)]
    for tree, vocab, kind, k, ke in cases:
        n = len(tree["parent"])
        logits_host = make_logits(rng, n, vocab, kind)["logits"]
        logits = dev_f32(logits_host)
        # a row stride of 4-element granularity is required by both entry points
        if vocab % 4:
            padded = torch.zeros((n, (vocab + 3) // 4 * 4), dtype=torch.float32, device=dev)
            padded[:, :vocab] = logits
            logits = padded[:, :vocab]
        tree_args = dict(parent=dev_i32(tree["parent"]), rank=dev_i32(tree["rank"]),
                         node_offsets=dev_i32([0, n]), root_token=dev_i32([17]))
        st = sage.new_status()
        want = sage.sage_expand_topk(logits, k, ke, status=st, **tree_args)
        got = sage.sage_expand_topk_static(logits, k, ke, out=_outputs(n, k, n, dev), status=st, **tree_args)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        assert torch.equal(got["topk_idx"], want["topk_idx"])
        assert torch.equal(got["draft_token"], want["draft_token"])
        for name in FLOAT_OUTPUTS:
            diff = (got[name].double() - want[name].double()).abs().max().item()
            assert diff <= ENTROPY_ABS, (name, diff)
        # and against the oracle itself, on the same logits
        check_logits({name: t.cpu().numpy() for name, t in got.items()}, logits_host, k, ke)


def test_static_scratch_rejects_problems_beyond_its_array_without_a_gpu():
    lib = sage.lib()
    fake = ctypes.c_void_p(0x1000)      # never dereferenced: the size check comes first
    rows = 8000                         # 8000 rows x 152 bytes of scratch each > 1 MiB
    assert sage.sage_expand_topk_workspace_size(rows, 152064) > sage.SAGE_STATIC_SCRATCH_BYTES
    code = lib.sage_expand_topk_static(fake, rows, 152064, 152064, 2, 2, fake, None, None, None, None, None,
                                       None, None, None, 0, None, None, None, None)
    assert code == sage.SAGE_ERR_TOO_LARGE
    assert "scratch" in sage.status_string(code)
    # the largest workload of this repository's benchmark fits with room to spare
    assert sage.sage_expand_topk_workspace_size(16 * 60, 152064) <= sage.SAGE_STATIC_SCRATCH_BYTES
