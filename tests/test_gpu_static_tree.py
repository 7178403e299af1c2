"""GPU parity on a second workload: a fixed-shape draft tree (the kind the paper compares its dynamic
tree with) through the mask, attention and acceptance steps.  Same bars as for the dynamic tree:
masks, position ids, accepted paths and extra tokens bit-exact (with the oracle's exemption margins
at temperature 1), attention within the bf16 tolerance."""
import numpy as np
import pytest
import torch

import paper_2406_16858_b200 as e2
from oracle import ref
from workloads import generators as gen
from workloads import static_tree

from harness import DEV, dev, gpu_accept, gpu_attention, host, new_status

pytestmark = pytest.mark.gpu

K, D = 10, static_tree.N_LEVELS


def _forest(B, V, seed):
    rng = np.random.default_rng(seed)
    R = ref.n_draft_rows(K, D)
    draft = (2.0 * rng.standard_normal((B, R, V))).astype(np.float32)
    draft[:, :, 7] += 6.0  # a likely token in every row: acceptance walks of several steps
    index, parent, depth, _, row_of = static_tree.shape(K)
    n = len(index)
    sel = ref.Selection(np.tile(index, (B, 1)), np.tile(parent, (B, 1)), static_tree.tokens(draft, K),
                        np.tile(depth, (B, 1)), np.full(B, n, np.int32))
    target = np.empty((B, n + 1, V), np.float32)
    for x in range(n + 1):
        row = 0 if x == 0 else int(row_of[x - 1])
        base = draft[:, row] if row >= 0 else (2.0 * rng.standard_normal((B, V))).astype(np.float32)
        target[:, x] = base + np.float32(0.5) * rng.standard_normal((B, V)).astype(np.float32)
    ua = rng.random((B, n), dtype=np.float32)
    ub = rng.random(B, dtype=np.float32)
    return draft, sel, target, ua, ub, n


@pytest.mark.parametrize("seed", range(3))
def test_mask_and_attention(seed):
    B, V = 3, 64
    _, sel, _, _, _, n = _forest(B, V, seed)
    kv_len = np.array([300, 0, 1025], np.int32)
    wbits, _, wpos, wst = ref.tree_mask(sel.parent, sel.depth, sel.n_sel, kv_len, n)
    bits = torch.zeros((B, n, 1), dtype=torch.int64, device=DEV)
    pos = torch.zeros((B, n), dtype=torch.int32, device=DEV)
    st = new_status()
    e2.tree_mask(dev(sel.parent), dev(sel.depth), dev(sel.n_sel), dev(kv_len), B, n, bits, None, pos, st)
    torch.cuda.synchronize()
    assert int(st.item()) == wst == 0
    assert (host(bits, np.uint64) == wbits).all() and (host(pos) == wpos).all()
    Hq, Hkv, d = 8, 2, 128
    rng = np.random.default_rng(seed + 50)
    kv_off = gen.kv_offsets(kv_len, n)
    rows = int(kv_off[-1] + kv_len[-1] + n)
    q = gen.f32_to_bf16_bits(rng.standard_normal((B, n, Hq, d)).astype(np.float32))
    kc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
    vc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
    got, _, st2 = gpu_attention(q, kc, vc, kv_off, kv_len, wbits, 1.0 / np.sqrt(d))
    _, want, _ = ref.tree_attention(q, kc, vc, kv_off, kv_len, wbits, 1.0 / np.sqrt(d), want_lse=True)
    assert st2 == 0
    assert np.abs(gen.bf16_bits_to_f32(got).astype(np.float64) - want).max() <= 2e-2


@pytest.mark.parametrize("temperature", [0.0, 1.0])
@pytest.mark.parametrize("V,seed", [(1000, 0), (1000, 1), (1000, 2), (32000, 3)])
def test_acceptance(temperature, V, seed):
    B = 16
    draft, sel, target, ua, ub, n = _forest(B, V, seed)
    d_arg = draft if temperature > 0 else None
    want = ref.accept(target, d_arg, sel, V, K, D, n, temperature, ua, ub, debug=temperature > 0)
    alen, apath, bonus, st = gpu_accept(target, d_arg, sel.index, sel.parent, sel.token, sel.n_sel, V, K, D, n,
                                        temperature, ua, ub)
    assert st == want.status == 0
    assert want.acc_len.max() >= 2  # the walks do get somewhere
    for b in range(B):
        if temperature > 0 and want.margins[b, 0] < 1e-6:
            continue
        assert alen[b] == want.acc_len[b] and (apath[b] == want.acc_path[b]).all()
        if temperature > 0 and want.margins[b, 1] < 1e-5:
            # a draw within 1e-5 of a step of the distribution function: a neighbour is acceptable
            # if its own step lies within that distance of the draw
            p = want.p_final[b]
            cdf = np.cumsum(p)
            thr, t = float(ub[b]) * cdf[-1], int(bonus[b])
            assert p[t] > 0 and cdf[t] - p[t] - 1e-5 * cdf[-1] <= thr <= cdf[t] + 1e-5 * cdf[-1]
            continue
        assert bonus[b] == want.bonus_token[b]
