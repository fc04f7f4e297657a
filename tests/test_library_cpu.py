"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header
declares, and rejects bad arguments on the host before touching a GPU."""
import ctypes
import os
import re

import paper_2602_00523_b200 as sage

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sage.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sage_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_symbols()
    assert {"sage_select_tree", "sage_expand_topk", "sage_tree_attention", "sage_accept",
            "sage_compact_kv"} <= set(names)
    lib = sage.lib()
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings():
    for code in (0, 1, 2, 3, 4, 5, 101, 102, 103, 104):
        assert sage.status_string(code) != "unknown status"
    assert sage.status_string(999) == "unknown status"


def test_workspace_queries():
    assert sage.sage_expand_topk_workspace_size(0, 100) == 0
    assert sage.sage_expand_topk_workspace_size(60, 152064) > 0
    one = sage.sage_tree_attention_workspace_size(1, 1, 60, 64, 8, 128, 257)
    assert one >= 60 * 64 * 130 * 4
    assert sage.sage_tree_attention_workspace_size(0, 1, 60, 64, 8, 128, 257) == 0


def test_host_side_argument_validation_needs_no_gpu():
    lib = sage.lib()
    fake = ctypes.c_void_p(0x1000)   # never dereferenced: the calls below fail validation first
    # null logits
    assert lib.sage_expand_topk(None, 4, 100, 100, 2, 2, fake, None, None, None, None, None, None, None, None, 0,
                                None, None, fake, 1 << 20, None, None) == sage.SAGE_ERR_INVALID_ARG
    # k above the supported maximum
    assert lib.sage_expand_topk(fake, 4, 1000, 1000, 17, 2, fake, None, None, None, None, None, None, None, None, 0,
                                None, None, fake, 1 << 20, None, None) == sage.SAGE_ERR_UNSUPPORTED
    # row stride not a multiple of 4 elements
    assert lib.sage_expand_topk(fake, 4, 1001, 1001, 2, 2, fake, None, None, None, None, None, None, None, None, 0,
                                None, None, fake, 1 << 20, None, None) == sage.SAGE_ERR_UNSUPPORTED
    # workspace too small
    assert lib.sage_expand_topk(fake, 4, 1000, 1000, 2, 2, fake, None, None, None, None, None, None, None, None, 0,
                                None, None, fake, 8, None, None) == sage.SAGE_ERR_WORKSPACE
    # attention: head_dim 64 unsupported, GQA group 3 unsupported, null q invalid
    args = [fake, fake, fake, 1 << 20, 1, 16, fake, 4, fake, fake, fake, 1, 8, 8, 2, 128, 64, 0.1, fake, fake,
            1 << 30, None, None]
    bad = list(args); bad[15] = 64
    assert lib.sage_tree_attention(*bad) == sage.SAGE_ERR_UNSUPPORTED
    bad = list(args); bad[13], bad[14] = 6, 2
    assert lib.sage_tree_attention(*bad) == sage.SAGE_ERR_UNSUPPORTED
    bad = list(args); bad[0] = None
    assert lib.sage_tree_attention(*bad) == sage.SAGE_ERR_INVALID_ARG
    bad = list(args); bad[16] = 16
    assert lib.sage_tree_attention(*bad) == sage.SAGE_ERR_UNSUPPORTED
    # accept / compact / select
    assert lib.sage_accept(fake, fake, fake, fake, 1, 0, fake, fake, fake, None, None) == sage.SAGE_ERR_INVALID_ARG
    assert lib.sage_compact_kv(fake, fake, 1 << 20, 1, 16, fake, 4, fake, fake, fake, 1, 8, 8, 64, 64, None,
                               None) == sage.SAGE_ERR_UNSUPPORTED
    pol = sage.make_policy([0.1, 0.4])          # ascending thresholds are rejected
    assert lib.sage_select_tree(fake, None, 1, ctypes.byref(pol), fake, None, None, None, None, None, None, None,
                                None, None, None) == sage.SAGE_ERR_INVALID_ARG
    pol = sage.make_policy([0.5])
    assert lib.sage_select_tree(fake, None, 0, ctypes.byref(pol), fake, None, None, None, None, None, None, None,
                                None, None, None) == sage.SAGE_OK      # empty batch: nothing to do


def test_grow_tree_argument_validation_needs_no_gpu():
    lib = sage.lib()
    fake = ctypes.c_void_p(0x1000)
    pol = sage.make_policy([])
    args = [fake, fake, 10, fake, None, 1, ctypes.byref(pol), 64, fake, fake, fake, fake, fake, fake, fake, None, None,
            None]
    bad = list(args); bad[2] = 17
    assert lib.sage_grow_tree(*bad) == sage.SAGE_ERR_UNSUPPORTED
    bad = list(args); bad[7] = 65
    assert lib.sage_grow_tree(*bad) == sage.SAGE_ERR_UNSUPPORTED
    bad = list(args); bad[0] = None
    assert lib.sage_grow_tree(*bad) == sage.SAGE_ERR_INVALID_ARG
    ok = list(args); ok[5] = 0
    assert lib.sage_grow_tree(*ok) == sage.SAGE_OK


def test_update_history_argument_validation_needs_no_gpu():
    lib = sage.lib()
    fake = ctypes.c_void_p(0x1000)
    pol = sage.make_history_policy()
    assert lib.sage_update_history(fake, 0, ctypes.byref(pol), fake, fake, fake, None, None) == sage.SAGE_OK
    assert lib.sage_update_history(None, 1, ctypes.byref(pol), fake, fake, fake, None, None) == sage.SAGE_ERR_INVALID_ARG
    bad = sage.make_history_policy(window=4, min_samples=5)
    assert lib.sage_update_history(fake, 1, ctypes.byref(bad), fake, fake, fake, None, None) == sage.SAGE_ERR_INVALID_ARG
    bad = sage.make_history_policy(lower=3.0, upper=2.0)
    assert lib.sage_update_history(fake, 1, ctypes.byref(bad), fake, fake, fake, None, None) == sage.SAGE_ERR_INVALID_ARG
