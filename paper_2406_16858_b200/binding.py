"""ctypes binding of ``libeagle2.so``: argument marshalling only.

Every function takes torch tensors that already live on the GPU (or raw integer addresses), passes
their ``data_ptr()`` and the current CUDA stream to the C entry point of the same name and raises
``Eagle2Error`` on a negative return code.  Nothing is computed here and there is no fallback: if the
library has not been built, importing this module's functions fails with instructions.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libeagle2.so")

OP_EXPAND, OP_RERANK, OP_TREE_MASK, OP_TREE_ATTENTION, OP_ACCEPT, OP_KV_COMPACT, OP_LM_HEAD_EXPAND = range(7)
STATUS_NONFINITE_LOGIT, STATUS_NOT_CLOSED, STATUS_KV_OVERFLOW = 1, 2, 4
STATUS_TIMEOUT, STATUS_BAD_TREE = 8, 32

EXPORTS = ("eagle2_version", "eagle2_strerror", "eagle2_workspace_bytes", "eagle2_workspace_init",
           "eagle2_expand", "eagle2_rerank", "eagle2_tree_mask", "eagle2_tree_attention",
           "eagle2_accept", "eagle2_kv_compact", "eagle2_expand_static", "eagle2_expand_variant",
           "eagle2_rerank_skipped", "eagle2_lm_head", "eagle2_set_wait_limit",
           "eagle2_tree_attention_launches", "eagle2_lm_head_expand", "eagle2_rerank_mask")
EXPAND_BY_CONFIDENCE = 1


class Eagle2Error(RuntimeError):
    def __init__(self, name: str, code: int):
        super().__init__(f"{name} failed with code {code}: {strerror(code)}")
        self.code = code


_lib = None


def lib_path() -> str:
    return _LIB_PATH


def lib() -> C.CDLL:
    """The loaded shared library (loads it on first use; never builds, never falls back)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with "
                              "`python -m paper_2406_16858_b200.build` (needs nvcc)")
        h = C.CDLL(_LIB_PATH)
        vp, i32, i64, sz, f32 = C.c_void_p, C.c_int, C.c_longlong, C.c_size_t, C.c_float
        h.eagle2_version.restype = i32
        h.eagle2_strerror.restype = C.c_char_p
        h.eagle2_strerror.argtypes = [i32]
        h.eagle2_workspace_bytes.restype = sz
        h.eagle2_workspace_bytes.argtypes = [i32] * 10
        h.eagle2_workspace_init.argtypes = [vp, sz, vp]
        h.eagle2_lm_head_expand.restype = i32
        h.eagle2_lm_head_expand.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        h.eagle2_tree_attention_launches.restype = i32
        h.eagle2_tree_attention_launches.argtypes = [i32] * 6
        h.eagle2_set_wait_limit.restype = i64
        h.eagle2_set_wait_limit.argtypes = [i64]
        h.eagle2_expand.argtypes = [vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        h.eagle2_expand_static.argtypes = [vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        h.eagle2_expand_static.restype = i32
        h.eagle2_expand_variant.argtypes = [vp, i64, i32, i32, i32, i32, i32, C.c_uint, vp, vp, vp, vp, vp, sz,
                                            vp, vp]
        h.eagle2_expand_variant.restype = i32
        h.eagle2_rerank.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        h.eagle2_lm_head.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
        h.eagle2_lm_head.restype = i32
        h.eagle2_rerank_skipped.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        h.eagle2_rerank_skipped.restype = i32
        h.eagle2_rerank_mask.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        h.eagle2_rerank_mask.restype = i32
        h.eagle2_tree_mask.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]
        h.eagle2_tree_attention.argtypes = [vp, vp, vp, i64, vp, vp, vp, i32, i32, i32, i32, i32, i32,
                                            f32, vp, vp, vp, sz, vp, vp]
        h.eagle2_accept.argtypes = [vp, i64, vp, i64, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32,
                                    vp, vp, vp, vp, vp, vp, sz, vp, vp]
        h.eagle2_kv_compact.argtypes = [vp, vp, i32, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp]
        for name in ("eagle2_workspace_init", "eagle2_expand", "eagle2_rerank", "eagle2_tree_mask",
                     "eagle2_tree_attention", "eagle2_accept", "eagle2_kv_compact"):
            getattr(h, name).restype = i32
        _lib = h
    return _lib


def version() -> int:
    return int(lib().eagle2_version())


def strerror(code: int) -> str:
    return lib().eagle2_strerror(int(code)).decode()


def _ptr(t) -> int | None:
    """Device address of a tensor (``None`` stays NULL; a plain int is passed through)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else 0
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(name: str, code: int) -> None:
    if code != 0:
        raise Eagle2Error(name, code)


def _ws(ws):
    if ws is None:
        return None, 0
    return ws.data_ptr(), ws.numel() * ws.element_size()


def workspace_bytes(op: int, B: int = 1, V: int = 1, k: int = 1, D: int = 1, m: int = 1, Hq: int = 1,
                    Hkv: int = 1, d: int = 128, max_kv_len: int = 0) -> int:
    return int(lib().eagle2_workspace_bytes(op, B, V, k, D, m, Hq, Hkv, d, max_kv_len))


def set_wait_limit(cycles: int) -> int:
    """Bound (SM clock cycles) of the device-side waits of later calls; <= 0 restores the default.
    Returns the bound that was in force."""
    return int(lib().eagle2_set_wait_limit(int(cycles)))


def tree_attention_launches(B: int, m: int, Hq: int, Hkv: int, d: int, max_kv_len: int) -> int:
    """Kernels one ``tree_attention`` call launches at these sizes."""
    return int(lib().eagle2_tree_attention_launches(B, m, Hq, Hkv, d, max_kv_len))


def workspace_init(ws, stream=None) -> None:
    p, n = _ws(ws)
    _check("eagle2_workspace_init", lib().eagle2_workspace_init(p, n, _stream(stream)))


def expand(draft_logits, batch_stride: int, B: int, V: int, k: int, D: int, s: int, tree_token,
           tree_parent, tree_value, frontier, ws, d_status, stream=None) -> None:
    p, n = _ws(ws)
    _check("eagle2_expand", lib().eagle2_expand(
        _ptr(draft_logits), batch_stride, B, V, k, D, s, _ptr(tree_token), _ptr(tree_parent),
        _ptr(tree_value), _ptr(frontier), p, n, _ptr(d_status), _stream(stream)))


def lm_head(hidden, weight, rows: int, H: int, V: int, logits, d_status, stream=None) -> None:
    """logits fp32 [rows, V] = hidden bf16 [rows, H] . weight bf16 [V, H]^T (the draft logits of ``expand``)."""
    _check("eagle2_lm_head", lib().eagle2_lm_head(_ptr(hidden), _ptr(weight), rows, H, V, _ptr(logits),
                                                  _ptr(d_status), _stream(stream)))


def lm_head_expand(hidden, weight, H: int, B: int, V: int, k: int, D: int, s: int, tree_token, tree_parent,
                   tree_value, frontier, ws, d_status, stream=None) -> None:
    """``lm_head`` and ``expand`` of one step in one pass over the weights (the logits are never written)."""
    p, n = _ws(ws)
    _check("eagle2_lm_head_expand", lib().eagle2_lm_head_expand(
        _ptr(hidden), _ptr(weight), H, B, V, k, D, s, _ptr(tree_token), _ptr(tree_parent), _ptr(tree_value),
        _ptr(frontier), p, n, _ptr(d_status), _stream(stream)))


def expand_variant(draft_logits, batch_stride: int, B: int, V: int, k: int, D: int, s: int, flags: int,
                   tree_token, tree_parent, tree_value, frontier, ws, d_status, stream=None) -> None:
    """``expand`` with a choice of what ranks the next frontier (``EXPAND_BY_CONFIDENCE``: a node's
    own log-probability instead of its value; stored values stay the path sums)."""
    p, n = _ws(ws)
    _check("eagle2_expand_variant", lib().eagle2_expand_variant(
        _ptr(draft_logits), batch_stride, B, V, k, D, s, flags, _ptr(tree_token), _ptr(tree_parent),
        _ptr(tree_value), _ptr(frontier), p, n, _ptr(d_status), _stream(stream)))


def expand_static(draft_logits, batch_stride: int, B: int, V: int, k: int, D: int, s: int, tree_token,
                  tree_parent, tree_value, frontier, d_status, stream=None) -> None:
    """``expand`` for callers that cannot allocate a workspace: the scratch is a fixed buffer inside
    the library (see the header for its size limit and the rule against overlapping calls)."""
    _check("eagle2_expand_static", lib().eagle2_expand_static(
        _ptr(draft_logits), batch_stride, B, V, k, D, s, _ptr(tree_token), _ptr(tree_parent),
        _ptr(tree_value), _ptr(frontier), _ptr(d_status), _stream(stream)))


def rerank(tree_token, tree_parent, tree_value, B: int, k: int, D: int, m: int, sel_index, sel_parent,
           sel_token, sel_depth, n_sel, d_status, stream=None) -> None:
    _check("eagle2_rerank", lib().eagle2_rerank(
        _ptr(tree_token), _ptr(tree_parent), _ptr(tree_value), B, k, D, m, _ptr(sel_index),
        _ptr(sel_parent), _ptr(sel_token), _ptr(sel_depth), _ptr(n_sel), _ptr(d_status),
        _stream(stream)))


def rerank_mask(tree_token, tree_parent, tree_value, kv_len, B: int, k: int, D: int, m: int, sel_index, sel_parent,
                sel_token, sel_depth, n_sel, mask_bits, mask_dense, pos_ids, d_status, stream=None) -> None:
    """``rerank`` and ``tree_mask`` in one launch."""
    _check("eagle2_rerank_mask", lib().eagle2_rerank_mask(
        _ptr(tree_token), _ptr(tree_parent), _ptr(tree_value), _ptr(kv_len), B, k, D, m, _ptr(sel_index),
        _ptr(sel_parent), _ptr(sel_token), _ptr(sel_depth), _ptr(n_sel), _ptr(mask_bits), _ptr(mask_dense),
        _ptr(pos_ids), _ptr(d_status), _stream(stream)))


def rerank_skipped(tree_token, tree_parent, tree_value, frontier, B: int, k: int, D: int, m: int, sel_index,
                   sel_parent, sel_token, sel_depth, n_sel, d_status, stream=None) -> None:
    """The selection without reranking: the frontier nodes of every expansion step, flattened."""
    _check("eagle2_rerank_skipped", lib().eagle2_rerank_skipped(
        _ptr(tree_token), _ptr(tree_parent), _ptr(tree_value), _ptr(frontier), B, k, D, m,
        _ptr(sel_index), _ptr(sel_parent), _ptr(sel_token), _ptr(sel_depth), _ptr(n_sel),
        _ptr(d_status), _stream(stream)))


def tree_mask(sel_parent, sel_depth, n_sel, kv_len, B: int, m: int, mask_bits, mask_dense, pos_ids,
              d_status, stream=None) -> None:
    _check("eagle2_tree_mask", lib().eagle2_tree_mask(
        _ptr(sel_parent), _ptr(sel_depth), _ptr(n_sel), _ptr(kv_len), B, m, _ptr(mask_bits),
        _ptr(mask_dense), _ptr(pos_ids), _ptr(d_status), _stream(stream)))


def tree_attention(q, k_cache, v_cache, cache_rows: int, kv_off, kv_len, mask_bits, B: int, m: int,
                   Hq: int, Hkv: int, d: int, max_kv_len: int, scale: float, out, lse, ws, d_status,
                   stream=None) -> None:
    p, n = _ws(ws)
    _check("eagle2_tree_attention", lib().eagle2_tree_attention(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), cache_rows, _ptr(kv_off), _ptr(kv_len), _ptr(mask_bits),
        B, m, Hq, Hkv, d, max_kv_len, scale, _ptr(out), _ptr(lse), p, n, _ptr(d_status),
        _stream(stream)))


def accept(target_logits, t_stride: int, draft_logits_all, d_stride: int, sel_index, sel_parent,
           sel_token, n_sel, B: int, V: int, k: int, D: int, m: int, temperature: float, u_accept,
           u_bonus, acc_len, acc_path, bonus_token, ws, d_status, stream=None) -> None:
    p, n = _ws(ws)
    _check("eagle2_accept", lib().eagle2_accept(
        _ptr(target_logits), t_stride, _ptr(draft_logits_all), d_stride, _ptr(sel_index),
        _ptr(sel_parent), _ptr(sel_token), _ptr(n_sel), B, V, k, D, m, temperature, _ptr(u_accept),
        _ptr(u_bonus), _ptr(acc_len), _ptr(acc_path), _ptr(bonus_token), p, n, _ptr(d_status),
        _stream(stream)))


def kv_compact(k_layers, v_layers, n_layers: int, kv_off, kv_len, acc_path, acc_len, B: int, m: int,
               D: int, Hkv: int, d: int, d_status, stream=None) -> None:
    """k_layers / v_layers: int64 device tensors holding the layers' cache base addresses."""
    _check("eagle2_kv_compact", lib().eagle2_kv_compact(
        _ptr(k_layers), _ptr(v_layers), n_layers, _ptr(kv_off), _ptr(kv_len), _ptr(acc_path),
        _ptr(acc_len), B, m, D, Hkv, d, _ptr(d_status), _stream(stream)))
