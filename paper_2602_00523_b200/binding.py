"""ctypes binding of libsage.so: argument marshalling only.

Every function below has the name of the C entry point it calls (include/sage.h),
takes torch CUDA tensors (PyTorch is used for device memory and streams, nothing
else), passes raw device pointers and sizes through the C ABI and returns the
output tensors.  Outputs and workspaces can be passed in (``out=`` dicts /
``ws=``) so that a caller can keep allocation out of its hot loop.  There is no
CPU fallback: if the shared library is missing, importing this module fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import torch

from .build import LIB_PATH

SAGE_OK = 0
SAGE_ERR_INVALID_ARG = 1
SAGE_ERR_UNSUPPORTED = 2
SAGE_ERR_WORKSPACE = 3
SAGE_ERR_CUDA = 4
SAGE_ERR_TOO_LARGE = 5
SAGE_STATIC_SCRATCH_BYTES = 1 << 20
SAGE_STATUS_BAD_TREE = 101
SAGE_STATUS_BAD_PAGE = 102
SAGE_STATUS_TIMEOUT = 103
SAGE_STATUS_BAD_PATH = 104
SAGE_MAX_NODES = 64
SAGE_MAX_TOPK = 16
SAGE_MAX_TEMPLATES = 8


class SagePolicy(ctypes.Structure):
    """Mirror of ``sage_tree_policy``."""
    _fields_ = [("n_templates", ctypes.c_int),
                ("alpha_thresholds", ctypes.c_float * SAGE_MAX_TEMPLATES),
                ("d_min", ctypes.c_float), ("d_max", ctypes.c_float),
                ("w_min", ctypes.c_float), ("w_max", ctypes.c_float)]


class SageHistoryPolicy(ctypes.Structure):
    """Mirror of ``sage_history_policy``."""
    _fields_ = [("window", ctypes.c_int), ("min_samples", ctypes.c_int),
                ("lower", ctypes.c_float), ("upper", ctypes.c_float), ("step", ctypes.c_float),
                ("d_lo", ctypes.c_float), ("d_hi", ctypes.c_float)]


class SageError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (code {code})")


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it first (python -m paper_2602_00523_b200.build); "
                      "this package has no fallback path")

_lib = ctypes.CDLL(LIB_PATH)
_vp, _i, _i64, _f, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t

_lib.sage_expand_topk.restype = _i
_lib.sage_expand_topk.argtypes = [_vp, _i, _i, _i64, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp,
                                  _vp, _vp, _vp, _i, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.sage_expand_topk_workspace_size.restype = _sz
_lib.sage_expand_topk_workspace_size.argtypes = [_i, _i]
_lib.sage_expand_topk_static.restype = _i
_lib.sage_expand_topk_static.argtypes = [_vp, _i, _i, _i64, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp,
                                         _vp, _vp, _vp, _i, _vp, _vp, _vp, _vp]
_lib.sage_select_tree.restype = _i
_lib.sage_select_tree.argtypes = [_vp, _vp, _i, ctypes.POINTER(SagePolicy), _vp, _vp, _vp,
                                  _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sage_grow_tree.restype = _i
_lib.sage_grow_tree.argtypes = [_vp, _vp, _i, _vp, _vp, _i, ctypes.POINTER(SagePolicy), _i,
                                _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sage_update_history.restype = _i
_lib.sage_update_history.argtypes = [_vp, _i, ctypes.POINTER(SageHistoryPolicy), _vp, _vp, _vp, _vp, _vp]
_lib.sage_build_ancestor_mask.restype = _i
_lib.sage_build_ancestor_mask.argtypes = [_vp, _vp, _i, _vp, _vp, _vp]
_lib.sage_tree_attention.restype = _i
_lib.sage_tree_attention.argtypes = [_vp, _vp, _vp, _i64, _i, _i, _vp, _i, _vp, _vp, _vp, _i, _i,
                                     _i, _i, _i, _i, _f, _vp, _vp, _sz, _vp, _vp]
_lib.sage_tree_attention_workspace_size.restype = _sz
_lib.sage_tree_attention_workspace_size.argtypes = [_i, _i, _i, _i, _i, _i, _i]
_lib.sage_accept.restype = _i
_lib.sage_accept.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp]
_lib.sage_compact_kv.restype = _i
_lib.sage_compact_kv.argtypes = [_vp, _vp, _i64, _i, _i, _vp, _i, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp]
_lib.sage_debug_attention_waits.restype = None
_lib.sage_debug_attention_waits.argtypes = [ctypes.c_longlong, _i]
_lib.sage_debug_attention_schedule.restype = None
_lib.sage_debug_attention_schedule.argtypes = [_i]
_lib.sage_status_string.restype = ctypes.c_char_p
_lib.sage_status_string.argtypes = [_i]


def lib() -> ctypes.CDLL:
    return _lib


def status_string(code: int) -> str:
    return _lib.sage_status_string(int(code)).decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device tensors only")
    if not t.is_contiguous():
        raise ValueError("contiguous tensors only")
    return t.data_ptr()


def _stream(stream) -> int:
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def _check(code: int, where: str):
    if code != SAGE_OK:
        raise SageError(code, where)


def make_policy(thresholds, d_min=3.0, d_max=8.0, w_min=2.0, w_max=10.0) -> SagePolicy:
    p = SagePolicy()
    p.n_templates = len(thresholds) + 1
    for j, t in enumerate(thresholds):
        p.alpha_thresholds[j] = float(t)
    p.d_min, p.d_max, p.w_min, p.w_max = d_min, d_max, w_min, w_max
    return p


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


def sage_expand_topk_workspace_size(rows: int, vocab: int) -> int:
    return int(_lib.sage_expand_topk_workspace_size(rows, vocab))


def sage_expand_topk(logits: torch.Tensor, k: int, k_entropy: int, *, parent=None, rank=None,
                     node_offsets=None, root_token=None, out: Optional[Dict[str, torch.Tensor]] = None,
                     ws: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                     stream=None) -> Dict[str, torch.Tensor]:
    """logits fp32 [rows, vocab] (row stride = logits.stride(0)).  Returns a dict with
    topk_idx, topk_logprob, entropy_full, entropy_topk, alpha, lse and, when the tree
    arrays are given, draft_token."""
    assert logits.dtype == torch.float32 and logits.dim() == 2 and logits.stride(1) == 1
    rows, vocab = logits.shape
    dev = logits.device
    o = {} if out is None else out
    o.setdefault("topk_idx", torch.empty((rows, k), dtype=torch.int32, device=dev))
    o.setdefault("topk_logprob", torch.empty((rows, k), dtype=torch.float32, device=dev))
    for name in ("entropy_full", "entropy_topk", "alpha", "lse"):
        o.setdefault(name, torch.empty(rows, dtype=torch.float32, device=dev))
    batch = 0
    if parent is not None:
        batch = node_offsets.numel() - 1
        o.setdefault("draft_token", torch.empty(parent.numel(), dtype=torch.int32, device=dev))
    if ws is None:
        ws = torch.empty(max(16, sage_expand_topk_workspace_size(rows, vocab)), dtype=torch.uint8, device=dev)
    code = _lib.sage_expand_topk(logits.data_ptr(), rows, vocab, logits.stride(0), k, k_entropy,
                                 _ptr(o["topk_idx"]), _ptr(o["topk_logprob"]), _ptr(o["entropy_full"]),
                                 _ptr(o["entropy_topk"]), _ptr(o["alpha"]), _ptr(o["lse"]),
                                 _ptr(parent), _ptr(rank), _ptr(node_offsets), batch, _ptr(root_token),
                                 _ptr(o.get("draft_token")), _ptr(ws), ws.numel(), _ptr(status), _stream(stream))
    _check(code, "sage_expand_topk")
    return o


def sage_expand_topk_static(logits: torch.Tensor, k: int, k_entropy: int, *, parent=None, rank=None,
                            node_offsets=None, root_token=None, out: Dict[str, torch.Tensor],
                            status: Optional[torch.Tensor] = None, stream=None) -> Dict[str, torch.Tensor]:
    """sage_expand_topk without a workspace argument, for callers that cannot allocate device
    memory: the scratch is an array inside the library.  To honour that, this wrapper
    allocates nothing either -- every output tensor must already be in ``out`` (topk_idx,
    topk_logprob, entropy_full, entropy_topk, alpha, lse, and draft_token when the tree
    arrays are given).  Calls on one GPU must not overlap; problems whose workspace would
    exceed SAGE_STATIC_SCRATCH_BYTES raise SageError(SAGE_ERR_TOO_LARGE)."""
    assert logits.dtype == torch.float32 and logits.dim() == 2 and logits.stride(1) == 1
    rows, vocab = logits.shape
    batch = node_offsets.numel() - 1 if parent is not None else 0
    code = _lib.sage_expand_topk_static(logits.data_ptr(), rows, vocab, logits.stride(0), k, k_entropy,
                                        _ptr(out["topk_idx"]), _ptr(out["topk_logprob"]),
                                        _ptr(out["entropy_full"]), _ptr(out["entropy_topk"]), _ptr(out["alpha"]),
                                        _ptr(out["lse"]), _ptr(parent), _ptr(rank), _ptr(node_offsets), batch,
                                        _ptr(root_token), _ptr(out.get("draft_token")), _ptr(status),
                                        _stream(stream))
    _check(code, "sage_expand_topk_static")
    return out


def sage_select_tree(alpha: torch.Tensor, policy: SagePolicy, *, alpha_row=None, batch: Optional[int] = None,
                     bank_parent=None, bank_rank=None, bank_n_nodes=None, handover: bool = False,
                     out: Optional[Dict[str, torch.Tensor]] = None, status=None, stream=None):
    """Returns template_id, depth_cont, width_cont (and next_parent / next_rank /
    next_node_offsets when ``handover``)."""
    dev = alpha.device
    if batch is None:
        batch = alpha_row.numel() if alpha_row is not None else alpha.numel()
    o = {} if out is None else out
    o.setdefault("template_id", torch.empty(batch, dtype=torch.int32, device=dev))
    o.setdefault("depth_cont", torch.empty(batch, dtype=torch.float32, device=dev))
    o.setdefault("width_cont", torch.empty(batch, dtype=torch.float32, device=dev))
    if handover:
        o.setdefault("next_parent", torch.full((batch * SAGE_MAX_NODES,), -1, dtype=torch.int32, device=dev))
        o.setdefault("next_rank", torch.zeros(batch * SAGE_MAX_NODES, dtype=torch.int32, device=dev))
        o.setdefault("next_node_offsets", torch.zeros(batch + 1, dtype=torch.int32, device=dev))
    code = _lib.sage_select_tree(_ptr(alpha), _ptr(alpha_row), batch, ctypes.byref(policy),
                                 _ptr(o["template_id"]), _ptr(o["depth_cont"]), _ptr(o["width_cont"]),
                                 _ptr(bank_parent), _ptr(bank_rank), _ptr(bank_n_nodes),
                                 _ptr(o.get("next_parent")), _ptr(o.get("next_rank")),
                                 _ptr(o.get("next_node_offsets")), _ptr(status), _stream(stream))
    _check(code, "sage_select_tree")
    return o


def sage_grow_tree(topk_idx: torch.Tensor, topk_logprob: torch.Tensor, alpha: torch.Tensor, policy: SagePolicy,
                   tree: Dict[str, torch.Tensor], *, alpha_row=None, n_max: int = SAGE_MAX_NODES, d_max_seq=None,
                   status=None, stream=None) -> Dict[str, torch.Tensor]:
    """One level of dynamic tree construction, in place on ``tree`` (parent, rank, depth, token:
    int32 [batch * SAGE_MAX_NODES]; cum_logprob fp32 of the same length; n_nodes, frontier_begin:
    int32 [batch]).  topk_idx / topk_logprob: [batch * SAGE_MAX_NODES, k]."""
    batch = tree["n_nodes"].numel()
    k = topk_idx.shape[1]
    code = _lib.sage_grow_tree(_ptr(topk_idx), _ptr(topk_logprob), k, _ptr(alpha), _ptr(alpha_row), batch,
                               ctypes.byref(policy), n_max, _ptr(tree["parent"]), _ptr(tree["rank"]),
                               _ptr(tree["depth"]), _ptr(tree["token"]), _ptr(tree["cum_logprob"]),
                               _ptr(tree["n_nodes"]), _ptr(tree["frontier_begin"]), _ptr(d_max_seq), _ptr(status),
                               _stream(stream))
    _check(code, "sage_grow_tree")
    return tree


def make_history_policy(window=10, min_samples=None, lower=2.0, upper=3.0, step=1.0, d_lo=3.0, d_hi=8.0):
    p = SageHistoryPolicy()
    p.window, p.min_samples = window, window if min_samples is None else min_samples
    p.lower, p.upper, p.step, p.d_lo, p.d_hi = lower, upper, step, d_lo, d_hi
    return p


def sage_update_history(path_len: torch.Tensor, policy: SageHistoryPolicy, window_buf: torch.Tensor,
                        count: torch.Tensor, d_max: torch.Tensor, *, status=None, stream=None):
    """In place: window_buf int32 [batch, window], count int32 [batch], d_max fp32 [batch]."""
    _check(_lib.sage_update_history(_ptr(path_len), path_len.numel(), ctypes.byref(policy), _ptr(window_buf),
                                    _ptr(count), _ptr(d_max), _ptr(status), _stream(stream)), "sage_update_history")
    return d_max


def sage_build_ancestor_mask(parent: torch.Tensor, node_offsets: torch.Tensor, *, out=None, status=None, stream=None):
    """Returns int64 [sum_nodes] holding the uint64 bitsets."""
    batch = node_offsets.numel() - 1
    anc = out if out is not None else torch.zeros(parent.numel(), dtype=torch.int64, device=parent.device)
    _check(_lib.sage_build_ancestor_mask(_ptr(parent), _ptr(node_offsets), batch, _ptr(anc), _ptr(status),
                                         _stream(stream)), "sage_build_ancestor_mask")
    return anc


def sage_tree_attention_workspace_size(n_layers, batch, sum_nodes, n_q_heads, n_kv_heads, head_dim, max_pages) -> int:
    return int(_lib.sage_tree_attention_workspace_size(n_layers, batch, sum_nodes, n_q_heads, n_kv_heads,
                                                       head_dim, max_pages))


def sage_tree_attention(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: torch.Tensor,
                        seq_len: torch.Tensor, parent: torch.Tensor, node_offsets: torch.Tensor, sm_scale: float,
                        *, out=None, ws=None, status=None, stream=None) -> torch.Tensor:
    """q bf16 [layers, sum_nodes, Hq, d]; pools bf16 [layers, pages, Hkv, P, d];
    page_table int32 [B, max_pages].  Returns bf16 [layers, sum_nodes, Hq, d]."""
    assert q.dtype == torch.bfloat16 and k_pool.dtype == torch.bfloat16 and v_pool.dtype == torch.bfloat16
    n_layers, sum_nodes, Hq, d = q.shape
    _, n_pages, Hkv, P, _ = k_pool.shape
    batch, max_pages = page_table.shape
    layer_stride = k_pool.stride(0) if n_layers > 1 else n_pages * Hkv * P * d
    assert v_pool.shape == k_pool.shape and (n_layers == 1 or v_pool.stride(0) == layer_stride)
    if out is None:
        out = torch.empty_like(q)
    need = sage_tree_attention_workspace_size(n_layers, batch, sum_nodes, Hq, Hkv, d, max_pages)
    if ws is None:
        ws = torch.empty(max(16, need), dtype=torch.uint8, device=q.device)
    code = _lib.sage_tree_attention(_ptr(q), k_pool.data_ptr(), v_pool.data_ptr(), layer_stride, n_layers, n_pages,
                                    _ptr(page_table), max_pages, _ptr(seq_len), _ptr(parent), _ptr(node_offsets),
                                    batch, sum_nodes, Hq, Hkv, d, P, float(sm_scale), _ptr(out), _ptr(ws),
                                    ws.numel(), _ptr(status), _stream(stream))
    _check(code, "sage_tree_attention")
    return out


def sage_debug_attention_waits(wait_cycles: int = 0, producer_off: bool = False) -> None:
    """Cycle budget of the attention kernel's on-device waits (0 = default) and, for tests of the
    time-out path, a switch that keeps its copy warp from issuing anything."""
    _lib.sage_debug_attention_waits(int(wait_cycles), 1 if producer_off else 0)


def sage_debug_attention_schedule(schedule: int = 0) -> None:
    """0: the library picks the attention schedule per launch; 1: streaming; 2: split; 3: streaming on two-block clusters."""
    _lib.sage_debug_attention_schedule(int(schedule))


def sage_accept(parent, draft_token, target_argmax, node_offsets, max_path: int, *, out=None, status=None, stream=None):
    batch = node_offsets.numel() - 1
    dev = parent.device
    o = {} if out is None else out
    o.setdefault("path", torch.empty((batch, max_path), dtype=torch.int32, device=dev))
    o.setdefault("path_len", torch.empty(batch, dtype=torch.int32, device=dev))
    o.setdefault("bonus_token", torch.empty(batch, dtype=torch.int32, device=dev))
    _check(_lib.sage_accept(_ptr(parent), _ptr(draft_token), _ptr(target_argmax), _ptr(node_offsets), batch, max_path,
                            _ptr(o["path"]), _ptr(o["path_len"]), _ptr(o["bonus_token"]), _ptr(status),
                            _stream(stream)), "sage_accept")
    return o


def sage_compact_kv(k_pool, v_pool, page_table, seq_len, path, path_len, *, status=None, stream=None):
    """In place on k_pool, v_pool ([layers, pages, Hkv, P, d] bf16) and seq_len."""
    n_layers, n_pages, Hkv, P, d = k_pool.shape
    batch, max_pages = page_table.shape
    max_path = path.shape[1]
    layer_stride = k_pool.stride(0) if n_layers > 1 else n_pages * Hkv * P * d
    _check(_lib.sage_compact_kv(k_pool.data_ptr(), v_pool.data_ptr(), layer_stride, n_layers, n_pages,
                                _ptr(page_table), max_pages, _ptr(seq_len), _ptr(path), _ptr(path_len), batch,
                                max_path, Hkv, d, P, _ptr(status), _stream(stream)), "sage_compact_kv")
