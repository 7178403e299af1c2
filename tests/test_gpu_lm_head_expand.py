"""GPU parity of ``eagle2_lm_head_expand`` - the LM head fused with the expansion (Section 4.1), the
logits never written - against the oracle's pipeline LM head -> expansion.

The device logits are fp32 sums of bf16 products (error of a few 1e-6 on logits of standard
deviation 2), so a sequence is exempt where the oracle shows that this error could decide: two of
a row's k+1 largest logits closer than 1e-4, or a frontier cut by less than 1e-4.  Exempt
sequences are counted and held to a ceiling; tokens, parents and frontier of all others must be
identical and values within 1e-3 (they carry the logits' error through the log-sum-exp)."""
import numpy as np
import pytest
import torch

import paper_2406_16858_b200 as e2
from oracle import ref
from workloads import generators as gen

from harness import DEV, dev, host, make_ws, new_status

pytestmark = pytest.mark.gpu


def _device_tree(hidden, wb, B, V, k, D, H):
    """hidden: bf16 bits [B, R, H].  Runs the D fused steps; returns (token, parent, value, frontier, status)."""
    N, R = k + (D - 1) * k * k, 1 + (D - 1) * k
    token = torch.full((B, N), -1, dtype=torch.int32, device=DEV)
    parent = torch.full((B, N), -2, dtype=torch.int32, device=DEV)
    value = torch.full((B, N), float("-inf"), dtype=torch.float64, device=DEV)
    frontier = torch.zeros((B, k), dtype=torch.int32, device=DEV)
    st = new_status()
    ws = make_ws(e2.workspace_bytes(e2.OP_LM_HEAD_EXPAND, B=B, V=V, k=k, D=D))
    tw = dev(wb)
    for s in range(D):
        lo, n_s = (0, 1) if s == 0 else (1 + (s - 1) * k, k)
        step = dev(np.ascontiguousarray(hidden[:, lo:lo + n_s]))  # [B][n_s][H]: the step's feature rows
        e2.lm_head_expand(step, tw, H, B, V, k, D, s, token, parent, value, frontier, ws, st)
    torch.cuda.synchronize()
    return host(token), host(parent), host(value), host(frontier), int(st.item())


def _decided_by_rounding(want_logits, tree, b, k, D):
    """True where the oracle's own numbers show a choice closer than 1e-4 for sequence b."""
    top = -np.sort(-want_logits[b], axis=1)[:, :k + 1]
    if (np.diff(-top, axis=1) < 1e-4).any():
        return True
    for s in range(D):
        base = 0 if s == 0 else k + (s - 1) * k * k
        v = -np.sort(-tree.value[b, base:base + (k if s == 0 else k * k)])
        if len(v) > k and v[k - 1] - v[k] < 1e-4:
            return True
    return False


@pytest.mark.parametrize("B,k,D,H,V", [
    (3, 4, 3, 128, 1000),      # a handful of rows: one row tile, four vocabulary tiles
    (1, 10, 2, 64, 200),       # a single vocabulary tile, a single partial per row
    (16, 10, 3, 256, 5000),    # 160 rows: two row tiles per pass
    (32, 10, 2, 128, 2049),    # 320 rows: two passes over the weights; ragged last vocabulary tile
    (9, 16, 2, 192, 3001),     # the widest list the fused path holds (k = 16), 144 rows
    (20, 7, 3, 64, 40000),     # more vocabulary tiles than blocks: every block folds two tiles or more
    (13, 10, 2, 64, 3000),     # 130 rows: a pair pass whose instruction width (144) is no multiple of 32
    (2, 4, 2, 64, 100),        # a vocabulary smaller than one tile
    (30, 10, 2, 64, 40000),    # 300 rows: a pass of block pairs, then 44 rows on single blocks (twice the producers per row)
])
def test_fused_tree_against_the_oracle_pipeline(B, k, D, H, V):
    R = 1 + (D - 1) * k
    checked = exempt = 0
    for seed in range(2):
        hb, wb = gen.lm_head_inputs(B * R, H, V, seed=7 * B + k + seed)
        hidden = hb.reshape(B, R, H)
        want_logits = ref.lm_head(hb, wb).reshape(B, R, V)
        tree = ref.build_tree(want_logits.astype(np.float32), V, k, D)
        tok, par, val, fr, st = _device_tree(hidden, wb, B, V, k, D, H)
        assert st == tree.status == 0
        for b in range(B):
            if _decided_by_rounding(want_logits, tree, b, k, D):
                exempt += 1
                continue
            checked += 1
            assert (tok[b] == tree.token[b]).all() and (par[b] == tree.parent[b]).all(), b
            assert np.abs(val[b] - tree.value[b]).max() < 1e-3
            assert (fr[b] == tree.frontier[b]).all()
    assert checked >= B  # most sequences are decided clearly ...
    # ... a near-tie is the exception, less so with many rows and wide lists: a sequence has up to
    # (1 + (D-1)k) * k gaps between neighbouring top logits, each below 1e-4 with probability ~1e-3
    assert exempt <= max(2, checked)


def test_full_vocabulary_of_the_llama3_shape():
    """The whole 128256-entry vocabulary (501 tiles over 148 blocks, 1480 keys per row for the merge)
    with 160 rows; the hidden size is kept small so that the oracle's LM head stays within seconds."""
    B, k, D, H, V = 16, 10, 2, 128, 128256
    R = 1 + (D - 1) * k
    hb, wb = gen.lm_head_inputs(B * R, H, V, seed=77)
    want_logits = ref.lm_head(hb, wb).reshape(B, R, V)
    tree = ref.build_tree(want_logits.astype(np.float32), V, k, D)
    tok, par, val, fr, st = _device_tree(hb.reshape(B, R, H), wb, B, V, k, D, H)
    assert st == 0
    checked = 0
    for b in range(B):
        if _decided_by_rounding(want_logits, tree, b, k, D):
            continue
        checked += 1
        assert (tok[b] == tree.token[b]).all() and (par[b] == tree.parent[b]).all()
        assert np.abs(val[b] - tree.value[b]).max() < 1e-3
        assert (fr[b] == tree.frontier[b]).all()
    assert checked >= B // 2


def test_fused_equals_the_two_separate_calls():
    """The same features through ``lm_head`` + ``expand``: identical tokens, parents and frontier
    wherever the separate path's own fp32 logits leave no near-tie."""
    B, k, D, H, V = 12, 10, 3, 128, 6000
    R = 1 + (D - 1) * k
    hb, wb = gen.lm_head_inputs(B * R, H, V, seed=5)
    tok, par, val, fr, st = _device_tree(hb.reshape(B, R, H), wb, B, V, k, D, H)
    assert st == 0
    logits = torch.zeros((B, R, V), dtype=torch.float32, device=DEV)
    st2 = new_status()
    e2.lm_head(dev(hb), dev(wb), B * R, H, V, logits, st2)
    torch.cuda.synchronize()
    tree = ref.build_tree(host(logits), V, k, D)  # the oracle on exactly the separate path's logits
    want64 = host(logits).astype(np.float64)
    same = 0
    for b in range(B):
        if _decided_by_rounding(want64, tree, b, k, D):
            continue
        same += 1
        assert (tok[b] == tree.token[b]).all() and (par[b] == tree.parent[b]).all()
        assert (fr[b] == tree.frontier[b]).all()
        assert np.abs(val[b] - tree.value[b]).max() < 1e-4
    assert same >= B // 2


def test_refusals_and_limits():
    hb, wb = gen.lm_head_inputs(4, 64, 100, seed=1)
    th, tw = dev(hb), dev(wb)
    N = 4 + 4 * 4
    tok = torch.zeros((1, N), dtype=torch.int32, device=DEV)
    val = torch.zeros((1, N), dtype=torch.float64, device=DEV)
    fr = torch.zeros((1, 4), dtype=torch.int32, device=DEV)
    st = new_status()
    ws = make_ws(e2.workspace_bytes(e2.OP_LM_HEAD_EXPAND, B=1, V=100, k=4, D=2))
    with pytest.raises(e2.Eagle2Error) as err:
        e2.lm_head_expand(th, tw, 48, 1, 100, 4, 2, 0, tok, tok, val, fr, ws, st)      # H not a multiple of 64
    assert err.value.code == -2
    with pytest.raises(e2.Eagle2Error) as err:
        e2.lm_head_expand(th, tw, 64, 1, 100, 17, 2, 0, tok, tok, val, fr, ws, st)     # k beyond the fused path's list
    assert err.value.code == -2
    with pytest.raises(e2.Eagle2Error) as err:
        e2.lm_head_expand(th, tw, 64, 1, 100, 4, 2, 0, tok, tok, val, fr, None, st)    # no workspace
    assert err.value.code == -4
    assert e2.workspace_bytes(e2.OP_LM_HEAD_EXPAND, B=1, V=100, k=17, D=2) == 0
