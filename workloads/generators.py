"""Seeded synthetic inputs (host side, numpy Philox) for the draft-and-verify hot path.

These stand in for the draft-model and target-model outputs on the paper's evaluation sets, which
are not available: only their shapes and a plausible value structure are reproduced.

Recipe
  draft row      = 2*N(0,1)^V  (fp32)  + a boost on one uniformly chosen "likely" token:
                   +8 when the row is "easy" (probability p_easy), +2 otherwise
  target row     = the draft row that expanded the node (a fresh draft-style row for a node that
                   was never expanded) + N(0, std 0.5)
  calibrated target row (acceptance-length studies only) = that same base row with one token
                   raised above all others, the token drawn from the base row's softmax by the
                   Gumbel-max trick: a greedy verifier then accepts a child with exactly the
                   probability the draft gave it
  LM head        feature rows ~ N(0,1), weight [V][H] ~ N(0, (2/sqrt(H))^2), both rounded to bf16:
                   logits of standard deviation 2 like the draft rows above (random weights of
                   the right shape; no trained head is available)
  Q, K, V        ~ N(0,1) rounded to bf16
  uniforms       ~ U[0,1) fp32
  ragged lengths = round(exp(U(ln lo, ln hi)))

Nothing here depends on the method: the only structural helper, ``node_draft_rows``, is the index
convention of the interface (which draft row expanded which node).
"""
from __future__ import annotations

import numpy as np

from .configs import Config


def rng_for(seed: int, stream: int) -> np.random.Generator:
    """Independent counter-based stream per (seed, purpose)."""
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream]))


STREAM_DRAFT, STREAM_TARGET, STREAM_FRESH, STREAM_QKV, STREAM_U, STREAM_LEN, STREAM_EASY = range(7)
STREAM_GUMBEL = 7
STREAM_LM_HEAD = 8


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    rounded = (u + (0x7FFF + ((u >> 16) & 1))) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def _boosted_rows(rng: np.random.Generator, n_rows: int, V: int, p_easy: float) -> np.ndarray:
    rows = (2.0 * rng.standard_normal((n_rows, V), dtype=np.float32)).astype(np.float32)
    likely = rng.integers(0, V, size=n_rows)
    easy = rng.random(n_rows) < p_easy
    rows[np.arange(n_rows), likely] += np.where(easy, 8.0, 2.0).astype(np.float32)
    return rows


def p_easy_per_sequence(cfg: Config, seed: int) -> np.ndarray:
    if cfg.p_easy is not None:
        return np.full(cfg.B, cfg.p_easy, np.float64)
    return rng_for(seed, STREAM_EASY).random(cfg.B)


def draft_rows(cfg: Config, seed: int) -> np.ndarray:
    """fp32 [B, R, V]: row 0 feeds expansion step 0, rows 1+(s-1)k+j feed frontier slot j of step s."""
    pe = p_easy_per_sequence(cfg, seed)
    out = np.empty((cfg.B, cfg.R, cfg.V), np.float32)
    for b in range(cfg.B):
        out[b] = _boosted_rows(rng_for(seed, STREAM_DRAFT * 1000003 + b), cfg.R, cfg.V, pe[b])
    return out


def node_draft_rows(tree_parent: np.ndarray, k: int, D: int) -> np.ndarray:
    """[B, N] draft row that expanded each candidate node, or -1 (index convention only: the
    children written by frontier slot j of step s all carry that slot's node as parent)."""
    B, N = tree_parent.shape
    rows = np.full((B, N), -1, np.int32)
    for s in range(1, D):
        for j in range(k):
            first_child = k + (s - 1) * k * k + j * k
            node = tree_parent[:, first_child]
            ok = node >= 0
            rows[np.arange(B)[ok], node[ok]] = 1 + (s - 1) * k + j
    return rows


def target_rows(cfg: Config, seed: int, draft: np.ndarray, tree_parent: np.ndarray,
                sel_index: np.ndarray) -> np.ndarray:
    """fp32 [B, m+1, V]: row 0 for the root, row 1+x for flat node x (padding rows get fresh rows)."""
    B, m, V = cfg.B, cfg.m, cfg.V
    nd = node_draft_rows(tree_parent, cfg.k, cfg.D)
    pe = p_easy_per_sequence(cfg, seed)
    out = np.empty((B, m + 1, V), np.float32)
    for b in range(B):
        fresh = rng_for(seed, STREAM_FRESH * 1000003 + b)
        noise = rng_for(seed, STREAM_TARGET * 1000003 + b)
        for r in range(m + 1):
            if r == 0:
                base = draft[b, 0]
            else:
                idx = int(sel_index[b, r - 1])
                row = int(nd[b, idx]) if idx >= 0 else -1
                base = draft[b, row] if row >= 0 else _boosted_rows(fresh, 1, V, pe[b])[0]
            out[b, r] = base + np.float32(0.5) * noise.standard_normal(V, dtype=np.float32)
    return out


def target_rows_calibrated(cfg: Config, seed: int, draft: np.ndarray, tree_parent: np.ndarray,
                           sel_index: np.ndarray) -> np.ndarray:
    """fp32 [B, m+1, V] like ``target_rows``, but the row's largest logit sits on a token drawn from
    the base row's own softmax (argmax of row + Gumbel noise), 4 above the previous maximum."""
    B, m, V = cfg.B, cfg.m, cfg.V
    nd = node_draft_rows(tree_parent, cfg.k, cfg.D)
    pe = p_easy_per_sequence(cfg, seed)
    out = np.empty((B, m + 1, V), np.float32)
    for b in range(B):
        fresh = rng_for(seed, STREAM_FRESH * 1000003 + b)
        gum = rng_for(seed, STREAM_GUMBEL * 1000003 + b)
        for r in range(m + 1):
            if r == 0:
                base = draft[b, 0]
            else:
                idx = int(sel_index[b, r - 1])
                row = int(nd[b, idx]) if idx >= 0 else -1
                base = draft[b, row] if row >= 0 else _boosted_rows(fresh, 1, V, pe[b])[0]
            drawn = int(np.argmax(base.astype(np.float64) + gum.gumbel(size=V)))
            out[b, r] = base
            out[b, r, drawn] = base.max() + np.float32(4.0)
    return out


def uniforms(cfg: Config, seed: int):
    """(u_accept fp32 [B,m], u_bonus fp32 [B]) in [0,1)."""
    rng = rng_for(seed, STREAM_U)
    return rng.random((cfg.B, cfg.m), dtype=np.float32), rng.random(cfg.B, dtype=np.float32)


def kv_lengths(cfg: Config, seed: int) -> np.ndarray:
    if cfg.kv_len_range is None:
        return np.full(cfg.B, cfg.kv_len, np.int32)
    lo, hi = cfg.kv_len_range
    u = rng_for(seed, STREAM_LEN).random(cfg.B)
    return np.rint(np.exp(np.log(lo) + u * (np.log(hi) - np.log(lo)))).astype(np.int32)


def kv_offsets(kv_len: np.ndarray, m: int, align: int = 1) -> np.ndarray:
    """Packed cache: sequence b owns rows kv_off[b] .. kv_off[b]+kv_len[b]+m-1."""
    span = kv_len.astype(np.int64) + m
    if align > 1:
        span = (span + align - 1) // align * align
    off = np.zeros(len(kv_len), np.int64)
    off[1:] = np.cumsum(span)[:-1]
    return off


def qkv_bf16(cfg: Config, seed: int, kv_len: np.ndarray, kv_off: np.ndarray, layer: int = 0):
    """(q, k_cache, v_cache) as uint16 bf16 bit patterns: q [B,m,Hq,d], caches [rows,Hkv,d]."""
    rng = rng_for(seed, STREAM_QKV * 1000003 + layer)
    rows = int(kv_off[-1] + kv_len[-1] + cfg.m)
    q = f32_to_bf16_bits(rng.standard_normal((cfg.B, cfg.m, cfg.Hq, cfg.d), dtype=np.float32))
    kc = f32_to_bf16_bits(rng.standard_normal((rows, cfg.Hkv, cfg.d), dtype=np.float32))
    vc = f32_to_bf16_bits(rng.standard_normal((rows, cfg.Hkv, cfg.d), dtype=np.float32))
    return q, kc, vc


def lm_head_inputs(rows: int, H: int, V: int, seed: int):
    """(hidden [rows,H], weight [V,H]) as uint16 bf16 bit patterns."""
    rng = rng_for(seed, STREAM_LM_HEAD)
    hidden = f32_to_bf16_bits(rng.standard_normal((rows, H), dtype=np.float32))
    weight = f32_to_bf16_bits(rng.standard_normal((V, H), dtype=np.float32) * np.float32(2.0 / np.sqrt(H)))
    return hidden, weight
