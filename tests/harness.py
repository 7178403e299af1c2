"""Helpers shared by the GPU parity tests: numpy <-> device marshalling around the C-ABI binding."""
from __future__ import annotations

import numpy as np
import torch

import paper_2406_16858_b200 as e2

DEV = "cuda:0"


def dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV)
    if a.dtype == np.uint64:
        return torch.from_numpy(a.view(np.int64)).to(DEV)
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def host(t: torch.Tensor, dtype=None) -> np.ndarray:
    a = t.detach().cpu().numpy()
    return a.view(dtype) if dtype is not None else a


def new_status() -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=DEV)


def make_ws(nbytes: int) -> torch.Tensor:
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=DEV)
    assert ws.data_ptr() % 256 == 0
    e2.workspace_init(ws)
    return ws


class GpuTree:
    def __init__(self, B, V, k, D):
        self.B, self.V, self.k, self.D = B, V, k, D
        N = k + (D - 1) * k * k
        self.N = N
        self.token = torch.full((B, N), -1, dtype=torch.int32, device=DEV)
        self.parent = torch.full((B, N), -2, dtype=torch.int32, device=DEV)
        self.value = torch.full((B, N), float("-inf"), dtype=torch.float64, device=DEV)
        self.frontier = torch.zeros((B, k), dtype=torch.int32, device=DEV)
        self.status = new_status()
        self.ws = make_ws(e2.workspace_bytes(e2.OP_EXPAND, B=B, V=V, k=k, D=D))

    def expand_all(self, draft_rows_dev: torch.Tensor, flags: int = 0):
        """draft_rows_dev: fp32 [B, R, V] on the device.  flags != 0 goes through the variant entry."""
        B, V, k, D = self.B, self.V, self.k, self.D
        R = 1 + (D - 1) * k
        assert draft_rows_dev.shape == (B, R, V) and draft_rows_dev.is_contiguous()
        for s in range(D):
            lo = 0 if s == 0 else 1 + (s - 1) * k
            ptr = draft_rows_dev.data_ptr() + lo * V * 4
            if flags:
                e2.expand_variant(ptr, R * V, B, V, k, D, s, flags, self.token, self.parent, self.value,
                                  self.frontier, self.ws, self.status)
            else:
                e2.expand(ptr, R * V, B, V, k, D, s, self.token, self.parent, self.value, self.frontier,
                          self.ws, self.status)
        torch.cuda.synchronize()
        return self


class GpuSelection:
    def __init__(self, tree_token, tree_parent, tree_value, B, k, D, m, kv_len=None, dense=False, one_launch=False):
        """one_launch: through eagle2_rerank_mask instead of eagle2_rerank + eagle2_tree_mask."""
        self.B, self.m = B, m
        z = lambda *shape: torch.zeros(shape, dtype=torch.int32, device=DEV)  # noqa: E731
        self.index, self.parent, self.token, self.depth = z(B, m), z(B, m), z(B, m), z(B, m)
        self.n_sel = z(B)
        self.status = new_status()
        W = (m + 63) // 64
        self.mask_bits = torch.zeros((B, m, W), dtype=torch.int64, device=DEV)
        self.mask_dense = torch.zeros((B, m, m), dtype=torch.uint8, device=DEV) if dense else None
        self.pos_ids = z(B, m)
        self.kv_len = kv_len if kv_len is not None else z(B)
        if one_launch:
            e2.rerank_mask(tree_token, tree_parent, tree_value, self.kv_len, B, k, D, m, self.index, self.parent,
                           self.token, self.depth, self.n_sel, self.mask_bits, self.mask_dense, self.pos_ids,
                           self.status)
        else:
            e2.rerank(tree_token, tree_parent, tree_value, B, k, D, m, self.index, self.parent, self.token,
                      self.depth, self.n_sel, self.status)
            e2.tree_mask(self.parent, self.depth, self.n_sel, self.kv_len, B, m, self.mask_bits,
                         self.mask_dense, self.pos_ids, self.status)
        torch.cuda.synchronize()


def gpu_attention(q, kc, vc, kv_off, kv_len, mask_bits, scale, want_lse=False):
    """All arguments numpy (bf16 as uint16 bits); returns (out bf16 bits [B,m,Hq,d], lse or None, status)."""
    B, m, Hq, d = q.shape
    Hkv = kc.shape[1]
    max_len = int(kv_len.max()) if len(kv_len) else 0
    tq, tk, tv = dev(q), dev(kc), dev(vc)
    out = torch.zeros((B, m, Hq, d), dtype=torch.int16, device=DEV)
    lse = torch.zeros((B, Hq, m), dtype=torch.float32, device=DEV) if want_lse else None
    st = new_status()
    ws = make_ws(e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=B, m=m, Hq=Hq, Hkv=Hkv, d=d,
                                    max_kv_len=max_len))
    e2.tree_attention(tq, tk, tv, kc.shape[0], dev(kv_off.astype(np.int64)), dev(kv_len.astype(np.int32)),
                      dev(mask_bits), B, m, Hq, Hkv, d, max_len, scale, out, lse, ws, st)
    torch.cuda.synchronize()
    return host(out, np.uint16), (host(lse) if want_lse else None), int(st.item())


def gpu_accept(target, draft, sel_index, sel_parent, sel_token, n_sel, V, k, D, m, temperature,
               u_accept=None, u_bonus=None, t_stride=None, d_stride=None):
    """numpy in, numpy out: (acc_len, acc_path, bonus_token, status)."""
    B = sel_index.shape[0]
    R = 1 + (D - 1) * k
    t_stride = (m + 1) * V if t_stride is None else t_stride
    d_stride = (R * V if draft is not None else 0) if d_stride is None else d_stride
    tt = dev(target)
    td = dev(draft) if draft is not None else None
    acc_len = torch.zeros(B, dtype=torch.int32, device=DEV)
    acc_path = torch.zeros((B, D), dtype=torch.int32, device=DEV)
    bonus = torch.zeros(B, dtype=torch.int32, device=DEV)
    st = new_status()
    ws = make_ws(e2.workspace_bytes(e2.OP_ACCEPT, B=B, V=V, k=k, D=D, m=m))
    e2.accept(tt, t_stride, td, d_stride, dev(sel_index), dev(sel_parent), dev(sel_token), dev(n_sel),
              B, V, k, D, m, float(temperature),
              dev(u_accept) if u_accept is not None else None,
              dev(u_bonus) if u_bonus is not None else None, acc_len, acc_path, bonus, ws, st)
    torch.cuda.synchronize()
    return host(acc_len), host(acc_path), host(bonus), int(st.item())
