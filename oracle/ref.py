"""numpy front end of the CPU oracle (``eagle2_ref.c``).

Test infrastructure only: the tests, the smoke check and the benchmark's CPU
baseline may import this module; the product package never does.  The module
compiles the C file with gcc on first use (``build()``) and marshals numpy
arrays into it; it contains no arithmetic of the method.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "eagle2_ref.c")
_LIB = os.path.join(_HERE, "libeagle2_ref.so")

ST_NONFINITE_LOGIT = 1
ST_NOT_CLOSED = 2
ST_KV_OVERFLOW = 4
ST_BAD_TREE = 32


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over independent sequences)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def num_threads() -> int:
    return int(lib().eagle2_ref_num_threads())


def set_threads(n: int) -> int:
    """Threads for the loops over independent units (timing only); returns the previous count."""
    return int(lib().eagle2_ref_set_threads(int(n)))


def n_nodes(k: int, D: int) -> int:
    return k + (D - 1) * k * k


def n_draft_rows(k: int, D: int) -> int:
    return 1 + (D - 1) * k


def _p(a, ctype):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be contiguous"
    return a.ctypes.data_as(C.POINTER(ctype))


def _check(code: int, name: str):
    if code != 0:
        raise ValueError(f"{name} returned {code}")


@dataclass
class Tree:
    token: np.ndarray  # [B,N] i32
    parent: np.ndarray  # [B,N] i32
    value: np.ndarray  # [B,N] f64 (log of the path product)
    frontier: np.ndarray  # [B,k] i32
    status: int = 0


def new_tree(B: int, k: int, D: int) -> Tree:
    N = n_nodes(k, D)
    return Tree(np.full((B, N), -1, np.int32), np.full((B, N), -2, np.int32),
                np.full((B, N), -np.inf, np.float64), np.zeros((B, k), np.int32))


def expand(tree: Tree, draft_logits: np.ndarray, V: int, k: int, D: int, s: int,
           batch_stride: int | None = None, by_confidence: bool = False) -> None:
    """draft_logits: fp32 [B, n_s, V] (n_s = 1 at s == 0, else k), or any buffer with batch_stride."""
    B = tree.token.shape[0]
    assert draft_logits.dtype == np.float32
    n_s = k if s else 1
    if batch_stride is None:
        assert draft_logits.size == B * n_s * V
        batch_stride = n_s * V
    st = np.zeros(1, np.int32)
    _check(lib().eagle2_expand_variant_ref(
        _p(draft_logits, C.c_float), C.c_longlong(batch_stride), B, V, k, D, s, int(by_confidence),
        _p(tree.token, C.c_int32), _p(tree.parent, C.c_int32), _p(tree.value, C.c_double),
        _p(tree.frontier, C.c_int32), _p(st, C.c_int32)), "eagle2_expand_variant_ref")
    tree.status |= int(st[0])


def build_tree(draft_rows: np.ndarray, V: int, k: int, D: int, by_confidence: bool = False) -> Tree:
    """Run all D expansion steps.  draft_rows: fp32 [B, R, V]; row 0 feeds step 0 and rows
    1+(s-1)k .. 1+sk-1 feed step s."""
    B = draft_rows.shape[0]
    R = n_draft_rows(k, D)
    assert draft_rows.shape == (B, R, V)
    tree = new_tree(B, k, D)
    for s in range(D):
        lo = 0 if s == 0 else 1 + (s - 1) * k
        flat = draft_rows.reshape(-1)[lo * V:]
        st = np.zeros(1, np.int32)
        if by_confidence:
            _check(lib().eagle2_expand_variant_ref(
                _p(flat, C.c_float), C.c_longlong(R * V), B, V, k, D, s, 1,
                _p(tree.token, C.c_int32), _p(tree.parent, C.c_int32), _p(tree.value, C.c_double),
                _p(tree.frontier, C.c_int32), _p(st, C.c_int32)), "eagle2_expand_variant_ref")
        else:
            _check(lib().eagle2_expand_ref(
                _p(flat, C.c_float), C.c_longlong(R * V), B, V, k, D, s,
                _p(tree.token, C.c_int32), _p(tree.parent, C.c_int32), _p(tree.value, C.c_double),
                _p(tree.frontier, C.c_int32), _p(st, C.c_int32)), "eagle2_expand_ref")
        tree.status |= int(st[0])
    return tree


@dataclass
class Selection:
    index: np.ndarray  # [B,m] candidate index (-1 padding)
    parent: np.ndarray  # [B,m] flat position of the parent (-1 root)
    token: np.ndarray  # [B,m]
    depth: np.ndarray  # [B,m] level-1
    n_sel: np.ndarray  # [B]
    status: int = 0


def rerank(token, parent, value, k: int, D: int, m: int) -> Selection:
    B = token.shape[0]
    sel = Selection(*(np.zeros((B, m), np.int32) for _ in range(4)), np.zeros(B, np.int32))
    st = np.zeros(1, np.int32)
    _check(lib().eagle2_rerank_ref(
        _p(np.ascontiguousarray(token, np.int32), C.c_int32),
        _p(np.ascontiguousarray(parent, np.int32), C.c_int32),
        _p(np.ascontiguousarray(value, np.float64), C.c_double), B, k, D, m,
        _p(sel.index, C.c_int32), _p(sel.parent, C.c_int32), _p(sel.token, C.c_int32),
        _p(sel.depth, C.c_int32), _p(sel.n_sel, C.c_int32), _p(st, C.c_int32)), "eagle2_rerank_ref")
    sel.status = int(st[0])
    return sel


def rerank_skipped(token, parent, value, frontier, k: int, D: int, m: int) -> Selection:
    """Section 5.2, the ablation without reranking: the expansion phase's own selection, flattened."""
    B = token.shape[0]
    sel = Selection(*(np.zeros((B, m), np.int32) for _ in range(4)), np.zeros(B, np.int32))
    st = np.zeros(1, np.int32)
    _check(lib().eagle2_rerank_skipped_ref(
        _p(np.ascontiguousarray(token, np.int32), C.c_int32),
        _p(np.ascontiguousarray(parent, np.int32), C.c_int32),
        _p(np.ascontiguousarray(value, np.float64), C.c_double),
        _p(np.ascontiguousarray(frontier, np.int32), C.c_int32), B, k, D, m,
        _p(sel.index, C.c_int32), _p(sel.parent, C.c_int32), _p(sel.token, C.c_int32),
        _p(sel.depth, C.c_int32), _p(sel.n_sel, C.c_int32), _p(st, C.c_int32)),
        "eagle2_rerank_skipped_ref")
    sel.status = int(st[0])
    return sel


def tree_mask(sel_parent, sel_depth, n_sel, kv_len, m: int, dense: bool = False):
    """Returns (mask_bits u64 [B,m,W], mask_dense u8 [B,m,m] or None, pos_ids i32 [B,m], status)."""
    B = sel_parent.shape[0]
    W = (m + 63) // 64
    bits = np.zeros((B, m, W), np.uint64)
    dn = np.zeros((B, m, m), np.uint8) if dense else None
    pos = np.zeros((B, m), np.int32)
    st = np.zeros(1, np.int32)
    _check(lib().eagle2_tree_mask_ref(
        _p(np.ascontiguousarray(sel_parent, np.int32), C.c_int32),
        _p(np.ascontiguousarray(sel_depth, np.int32), C.c_int32),
        _p(np.ascontiguousarray(n_sel, np.int32), C.c_int32),
        _p(np.ascontiguousarray(kv_len, np.int32), C.c_int32), B, m,
        _p(bits, C.c_uint64), _p(dn, C.c_uint8), _p(pos, C.c_int32), _p(st, C.c_int32)),
        "eagle2_tree_mask_ref")
    return bits, dn, pos, int(st[0])


def tree_attention(q, k_cache, v_cache, kv_off, kv_len, mask_bits, scale: float, samples=None,
                   want_lse: bool = False):
    """q: uint16 (bf16 bits) [B,m,Hq,d]; k_cache/v_cache: uint16 [rows,Hkv,d].
    Returns (out bf16-bits, out f64, lse or None); indexed [B,m,Hq,d] / [B,Hq,m], or by sample
    when ``samples`` (int32 [n,3] of (b, head, query)) is given."""
    B, m, Hq, d = q.shape
    Hkv = k_cache.shape[1]
    assert q.dtype == np.uint16 and k_cache.dtype == np.uint16 and v_cache.dtype == np.uint16
    kv_off = np.ascontiguousarray(kv_off, np.int64)
    kv_len = np.ascontiguousarray(kv_len, np.int32)
    if samples is not None:
        samples = np.ascontiguousarray(samples, np.int32)
        n = samples.shape[0]
        out = np.zeros((n, d), np.uint16)
        out64 = np.zeros((n, d), np.float64)
        lse = np.zeros(n, np.float64) if want_lse else None
    else:
        n = 0
        out = np.zeros((B, m, Hq, d), np.uint16)
        out64 = np.zeros((B, m, Hq, d), np.float64)
        lse = np.zeros((B, Hq, m), np.float64) if want_lse else None
    st = np.zeros(1, np.int32)
    _check(lib().eagle2_tree_attention_ref(
        _p(q, C.c_uint16), _p(k_cache, C.c_uint16), _p(v_cache, C.c_uint16),
        _p(kv_off, C.c_int64), _p(kv_len, C.c_int32),
        _p(np.ascontiguousarray(mask_bits, np.uint64), C.c_uint64), B, m, Hq, Hkv, d,
        C.c_double(scale), _p(samples, C.c_int32), n, _p(out, C.c_uint16), _p(out64, C.c_double),
        _p(lse, C.c_double), _p(st, C.c_int32)), "eagle2_tree_attention_ref")
    return out, out64, lse


@dataclass
class Accepted:
    acc_len: np.ndarray  # [B]
    acc_path: np.ndarray  # [B,D] flat positions, -1 padded
    bonus_token: np.ndarray  # [B]
    margins: np.ndarray  # [B,2]: min |u-a|, relative CDF margin of the extra token
    accept_prob: np.ndarray | None = None  # [B,m] acceptance probability of each tested child
    p_final: np.ndarray | None = None  # [B,V] distribution the extra token is drawn from
    status: int = 0


def accept(target_logits, draft_logits_all, sel: Selection, V: int, k: int, D: int, m: int,
           temperature: float, u_accept=None, u_bonus=None, t_stride: int | None = None,
           d_stride: int | None = None, debug: bool = False) -> Accepted:
    """target_logits fp32 [B,m+1,V] (or shared with t_stride=0); draft_logits_all fp32 [B,R,V] or
    None (greedy, or the point-mass proposal at temperature > 0)."""
    B = sel.index.shape[0]
    assert target_logits.dtype == np.float32
    if t_stride is None:
        t_stride = (m + 1) * V
    if draft_logits_all is not None:
        assert draft_logits_all.dtype == np.float32
        if d_stride is None:
            d_stride = n_draft_rows(k, D) * V
    else:
        d_stride = 0
    out = Accepted(np.zeros(B, np.int32), np.zeros((B, D), np.int32), np.zeros(B, np.int32),
                   np.zeros((B, 2), np.float64))
    if debug:
        out.accept_prob = np.zeros((B, m), np.float64)
        out.p_final = np.zeros((B, V), np.float64)
    st = np.zeros(1, np.int32)
    ua = None if u_accept is None else np.ascontiguousarray(u_accept, np.float32)
    ub = None if u_bonus is None else np.ascontiguousarray(u_bonus, np.float32)
    _check(lib().eagle2_accept_ref(
        _p(target_logits, C.c_float), C.c_longlong(t_stride), _p(draft_logits_all, C.c_float),
        C.c_longlong(d_stride), _p(sel.index, C.c_int32), _p(sel.parent, C.c_int32),
        _p(sel.token, C.c_int32), _p(sel.n_sel, C.c_int32), B, V, k, D, m,
        C.c_double(temperature), _p(ua, C.c_float), _p(ub, C.c_float),
        _p(out.acc_len, C.c_int32), _p(out.acc_path, C.c_int32), _p(out.bonus_token, C.c_int32),
        _p(out.margins, C.c_double), _p(out.accept_prob, C.c_double), _p(out.p_final, C.c_double),
        _p(st, C.c_int32)), "eagle2_accept_ref")
    out.status = int(st[0])
    return out


def kv_compact(k_layers, v_layers, kv_off, kv_len, acc_path, acc_len, m: int, D: int) -> int:
    """k_layers/v_layers: lists of uint16 arrays [rows,Hkv,d], modified in place; kv_len in place."""
    n_layers = len(k_layers)
    B = len(kv_len)
    Hkv, d = k_layers[0].shape[1:] if n_layers else (1, 1)
    PtrArr = C.POINTER(C.c_uint16) * max(n_layers, 1)
    kp = PtrArr(*[_p(a, C.c_uint16) for a in k_layers])
    vp = PtrArr(*[_p(a, C.c_uint16) for a in v_layers])
    assert kv_len.dtype == np.int32 and kv_len.flags["C_CONTIGUOUS"]
    st = np.zeros(1, np.int32)
    _check(lib().eagle2_kv_compact_ref(
        kp, vp, n_layers, _p(np.ascontiguousarray(kv_off, np.int64), C.c_int64),
        _p(kv_len, C.c_int32), _p(np.ascontiguousarray(acc_path, np.int32), C.c_int32),
        _p(np.ascontiguousarray(acc_len, np.int32), C.c_int32), B, m, D, Hkv, d,
        _p(st, C.c_int32)), "eagle2_kv_compact_ref")
    return int(st[0])


def lm_head(hidden: np.ndarray, weight: np.ndarray) -> np.ndarray:
    """hidden uint16 (bf16 bits) [rows, H], weight uint16 [V, H] -> logits float64 [rows, V]."""
    assert hidden.dtype == np.uint16 and weight.dtype == np.uint16 and hidden.shape[1] == weight.shape[1]
    rows, H = hidden.shape
    V = weight.shape[0]
    out = np.zeros((rows, V), np.float64)
    _check(lib().eagle2_lm_head_ref(_p(np.ascontiguousarray(hidden), C.c_uint16),
                                    _p(np.ascontiguousarray(weight), C.c_uint16), rows, H, V,
                                    _p(out, C.c_double)), "eagle2_lm_head_ref")
    return out
