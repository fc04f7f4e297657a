"""B200-native (sm_100a) kernels for the data-parallel hot path of a SAGE decode
round: fused softmax-entropy + top-k, entropy -> tree template, tree-masked
verification attention over a paged bf16 KV cache, greedy acceptance and KV
compaction.  The product is the C-ABI library ``libsage.so`` (include/sage.h);
this package is its thin ctypes binding.  Build it with
``python -m paper_2602_00523_b200.build``.

The binding is loaded on first use of any of its names, so that the ``build``
submodule can be imported before the library exists; using a binding name while
the library is missing raises ImportError (there is no fallback path).
"""
import importlib

_BINDING_NAMES = (
    "SageError", "SagePolicy", "make_policy", "new_status", "status_string", "lib",
    "sage_expand_topk", "sage_expand_topk_workspace_size", "sage_expand_topk_static", "sage_select_tree",
    "sage_build_ancestor_mask", "sage_grow_tree", "sage_update_history", "make_history_policy",
    "SageHistoryPolicy", "sage_tree_attention", "sage_tree_attention_workspace_size",
    "sage_accept", "sage_compact_kv", "sage_debug_attention_waits", "sage_debug_attention_schedule",
    "SAGE_OK", "SAGE_ERR_INVALID_ARG", "SAGE_ERR_UNSUPPORTED", "SAGE_ERR_WORKSPACE", "SAGE_ERR_CUDA",
    "SAGE_ERR_TOO_LARGE", "SAGE_STATIC_SCRATCH_BYTES",
    "SAGE_STATUS_BAD_TREE", "SAGE_STATUS_BAD_PAGE", "SAGE_STATUS_TIMEOUT", "SAGE_STATUS_BAD_PATH",
    "SAGE_MAX_NODES", "SAGE_MAX_TOPK", "SAGE_MAX_TEMPLATES",
)
__all__ = list(_BINDING_NAMES)


def __getattr__(name):
    if name in _BINDING_NAMES:
        binding = importlib.import_module(".binding", __name__)
        for n in _BINDING_NAMES:
            globals()[n] = getattr(binding, n)
        return globals()[name]
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
