"""One draft-and-verify cycle as a fixed sequence of C-ABI calls on caller-owned device buffers.

``CycleBuffers`` owns the device tensors of one batch of sequences (tree arrays, selection, mask,
acceptance results, workspaces) and ``enqueue_cycle`` issues the launches of one cycle on the current
stream: D x expand, rerank, tree mask, one tree attention per layer, accept, KV compaction.  Nothing
synchronises, so the whole cycle can be captured in a CUDA graph.  This module only marshals
arguments; every step runs in the library's kernels.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import binding as e2


@dataclass
class CycleShape:
    B: int
    V: int
    k: int
    D: int
    m: int
    n_layers: int
    Hq: int
    Hkv: int
    d: int
    max_kv_len: int
    temperature: float

    @property
    def N(self) -> int:
        return self.k + (self.D - 1) * self.k * self.k

    @property
    def R(self) -> int:
        return 1 + (self.D - 1) * self.k


class CycleBuffers:
    def __init__(self, shape: CycleShape, device: torch.device | str = "cuda"):
        s, dev = shape, torch.device(device)
        self.shape, self.device = s, dev
        i32 = dict(dtype=torch.int32, device=dev)
        self.tree_token = torch.zeros((s.B, s.N), **i32)
        self.tree_parent = torch.zeros((s.B, s.N), **i32)
        self.tree_value = torch.zeros((s.B, s.N), dtype=torch.float64, device=dev)
        self.frontier = torch.zeros((s.B, s.k), **i32)
        self.sel_index = torch.zeros((s.B, s.m), **i32)
        self.sel_parent = torch.zeros((s.B, s.m), **i32)
        self.sel_token = torch.zeros((s.B, s.m), **i32)
        self.sel_depth = torch.zeros((s.B, s.m), **i32)
        self.n_sel = torch.zeros(s.B, **i32)
        self.mask_bits = torch.zeros((s.B, s.m, (s.m + 63) // 64), dtype=torch.int64, device=dev)
        self.pos_ids = torch.zeros((s.B, s.m), **i32)
        self.acc_len = torch.zeros(s.B, **i32)
        self.acc_path = torch.zeros((s.B, s.D), **i32)
        self.bonus_token = torch.zeros(s.B, **i32)
        self.status = torch.zeros(1, **i32)
        need = max(
            e2.workspace_bytes(e2.OP_EXPAND, B=s.B, V=s.V, k=s.k, D=s.D, m=s.m),
            e2.workspace_bytes(e2.OP_ACCEPT, B=s.B, V=s.V, k=s.k, D=s.D, m=s.m),
            e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=s.B, m=s.m, Hq=s.Hq, Hkv=s.Hkv, d=s.d,
                               max_kv_len=s.max_kv_len), 256)
        self.ws = torch.empty(need, dtype=torch.uint8, device=dev)
        e2.workspace_init(self.ws)

    # ---- the individual steps (all asynchronous on the current stream) -------------------------
    def expand_all(self, draft_rows: torch.Tensor) -> None:
        """draft_rows: fp32 [B, R, V]."""
        s = self.shape
        for step in range(s.D):
            lo = 0 if step == 0 else 1 + (step - 1) * s.k
            e2.expand(draft_rows.data_ptr() + lo * s.V * 4, s.R * s.V, s.B, s.V, s.k, s.D, step,
                      self.tree_token, self.tree_parent, self.tree_value, self.frontier, self.ws,
                      self.status)

    def rerank_and_mask(self, kv_len: torch.Tensor) -> None:
        s = self.shape
        e2.rerank_mask(self.tree_token, self.tree_parent, self.tree_value, kv_len, s.B, s.k, s.D, s.m,
                       self.sel_index, self.sel_parent, self.sel_token, self.sel_depth, self.n_sel,
                       self.mask_bits, None, self.pos_ids, self.status)

    def attention(self, q, k_cache, v_cache, kv_off, kv_len, out, scale: float) -> None:
        s = self.shape
        e2.tree_attention(q, k_cache, v_cache, k_cache.shape[0], kv_off, kv_len, self.mask_bits, s.B,
                          s.m, s.Hq, s.Hkv, s.d, s.max_kv_len, scale, out, None, self.ws, self.status)

    def accept(self, target_logits, draft_rows, u_accept, u_bonus) -> None:
        s = self.shape
        sampling = s.temperature > 0
        e2.accept(target_logits, (s.m + 1) * s.V, draft_rows if sampling else None,
                  s.R * s.V if sampling else 0, self.sel_index, self.sel_parent, self.sel_token,
                  self.n_sel, s.B, s.V, s.k, s.D, s.m, s.temperature, u_accept, u_bonus, self.acc_len,
                  self.acc_path, self.bonus_token, self.ws, self.status)

    def kv_compact(self, k_ptrs, v_ptrs, kv_off, kv_len) -> None:
        s = self.shape
        e2.kv_compact(k_ptrs, v_ptrs, s.n_layers, kv_off, kv_len, self.acc_path, self.acc_len, s.B,
                      s.m, s.D, s.Hkv, s.d, self.status)

    def launches_per_cycle(self) -> int:
        """Kernel launches of this library in one cycle (for bookkeeping in benchmarks)."""
        s = self.shape
        per_layer = e2.tree_attention_launches(s.B, s.m, s.Hq, s.Hkv, s.d, s.max_kv_len)
        return s.D + 1 + s.n_layers * per_layer + (2 if s.temperature > 0 else 1) + 2


def enqueue_cycle(buf: CycleBuffers, draft_rows, target_logits, u_accept, u_bonus, q_layers, k_layers,
                  v_layers, out_layers, k_ptrs, v_ptrs, kv_off, kv_len, scale: float) -> None:
    """One full cycle on the current stream.  q_layers/k_layers/v_layers/out_layers: per-layer tensors;
    k_ptrs/v_ptrs: int64 device tensors with the caches' base addresses."""
    buf.expand_all(draft_rows)
    buf.rerank_and_mask(kv_len)
    for q, kc, vc, out in zip(q_layers, k_layers, v_layers, out_layers):
        buf.attention(q, kc, vc, kv_off, kv_len, out, scale)
    buf.accept(target_logits, draft_rows, u_accept, u_bonus)
    buf.kv_compact(k_ptrs, v_ptrs, kv_off, kv_len)
