"""Pins for the oracle's tree-masked attention: dense numpy softmax, closed forms, a library causal
attention for the chain special case, and permutation invariance over cache rows."""
import numpy as np
import pytest
import torch

from oracle import ref
from workloads import generators as gen


def _case(seed, B, m, Hq, Hkv, d, lens, tree="random"):
    rng = np.random.default_rng(seed)
    kv_len = np.array(lens, np.int32)
    kv_off = gen.kv_offsets(kv_len, m)
    rows = int(kv_off[-1] + kv_len[-1] + m)
    q = gen.f32_to_bf16_bits(rng.standard_normal((B, m, Hq, d)).astype(np.float32))
    kc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
    vc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
    parent = np.full((B, m), -1, np.int32)
    depth = np.zeros((B, m), np.int32)
    for b in range(B):
        for i in range(m):
            if tree == "chain":
                parent[b, i] = i - 1
            elif i > 0:
                parent[b, i] = rng.integers(-1, i)
            depth[b, i] = 0 if parent[b, i] < 0 else depth[b, parent[b, i]] + 1
    bits, dense, _, st = ref.tree_mask(parent, depth, np.full(B, m, np.int32), kv_len, m, dense=True)
    assert st == 0
    return q, kc, vc, kv_off, kv_len, bits, dense


def _dense_numpy(q, kc, vc, kv_off, kv_len, dense, scale):
    B, m, Hq, d = q.shape
    Hkv = kc.shape[1]
    g = Hq // Hkv
    qf, kf, vf = (gen.bf16_bits_to_f32(x).astype(np.float64) for x in (q, kc, vc))
    out = np.zeros((B, m, Hq, d))
    for b in range(B):
        L = int(kv_len[b])
        ks = kf[kv_off[b]:kv_off[b] + L + m]
        vs = vf[kv_off[b]:kv_off[b] + L + m]
        vis = np.concatenate([np.ones((m, L), bool), dense[b].astype(bool)], axis=1)  # [m, L+m]
        for h in range(Hq):
            s = scale * qf[b, :, h] @ ks[:, h // g].T
            s = np.where(vis, s, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            out[b, :, h] = p @ vs[:, h // g]
    return out


@pytest.mark.parametrize("Hq,Hkv,d,lens", [(4, 4, 64, [37]), (8, 2, 32, [5, 0, 19]), (4, 1, 128, [64])])
def test_matches_dense_masked_softmax(Hq, Hkv, d, lens):
    m = 11
    q, kc, vc, off, kl, bits, dense = _case(2, len(lens), m, Hq, Hkv, d, lens)
    scale = 1.0 / np.sqrt(d)
    o16, o64, lse = ref.tree_attention(q, kc, vc, off, kl, bits, scale, want_lse=True)
    want = _dense_numpy(q, kc, vc, off, kl, dense, scale)
    np.testing.assert_allclose(o64, want, rtol=0, atol=1e-12)
    assert (o16 == gen.f32_to_bf16_bits(o64.astype(np.float32))).all()
    # sampled form returns the same numbers
    samples = np.array([[0, 1, 3], [len(lens) - 1, Hq - 1, m - 1]], np.int32)
    s16, s64, slse = ref.tree_attention(q, kc, vc, off, kl, bits, scale, samples=samples, want_lse=True)
    for t, (b, h, i) in enumerate(samples):
        assert (s64[t] == o64[b, i, h]).all() and slse[t] == lse[b, h, i]


def test_equal_keys_give_mean_of_visible_values():
    m, Hq, d, L = 7, 2, 16, 9
    q, kc, vc, off, kl, bits, dense = _case(4, 1, m, Hq, Hq, d, [L])
    kc[:] = kc[0, 0]  # every key identical -> uniform softmax over visible keys
    _, o64, _ = ref.tree_attention(q, kc, vc, off, kl, bits, 0.3)
    vf = gen.bf16_bits_to_f32(vc).astype(np.float64)
    for i in range(m):
        vis = list(range(L)) + [L + j for j in range(m) if dense[0, i, j]]
        for h in range(Hq):
            np.testing.assert_allclose(o64[0, i, h], vf[vis, h].mean(axis=0), atol=1e-12)


def test_chain_without_cache_is_causal_attention():
    m, H, d = 12, 3, 32
    q, kc, vc, off, kl, bits, _ = _case(6, 1, m, H, H, d, [0], tree="chain")
    scale = 1.0 / np.sqrt(d)
    _, o64, _ = ref.tree_attention(q, kc, vc, off, kl, bits, scale)
    tq, tk, tv = (torch.from_numpy(gen.bf16_bits_to_f32(x).astype(np.float64)) for x in (q, kc, vc))
    lib = torch.nn.functional.scaled_dot_product_attention(
        tq[0].permute(1, 0, 2), tk.permute(1, 0, 2), tv.permute(1, 0, 2), is_causal=True)
    np.testing.assert_allclose(o64[0], lib.permute(1, 0, 2).numpy(), atol=1e-12)


def test_dominant_key_selects_its_value_and_cache_permutation_is_invariant():
    m, H, d, L = 5, 2, 16, 20
    q, kc, vc, off, kl, bits, _ = _case(8, 1, m, H, H, d, [L])
    _, base, _ = ref.tree_attention(q, kc, vc, off, kl, bits, 0.25)
    perm = np.random.default_rng(0).permutation(L)
    kc2, vc2 = kc.copy(), vc.copy()
    kc2[:L], vc2[:L] = kc[perm], vc[perm]
    _, shuffled, _ = ref.tree_attention(q, kc2, vc2, off, kl, bits, 0.25)
    np.testing.assert_allclose(shuffled, base, atol=1e-13)
    # a huge scale makes the best-scoring visible key take all the weight
    _, sharp, _ = ref.tree_attention(q, kc, vc, off, kl, bits, 1e4)
    qf, kf, vf = (gen.bf16_bits_to_f32(x).astype(np.float64) for x in (q, kc, vc))
    scores = qf[0, 0, 0] @ kf[:L + 1, 0].T  # query 0 sees the cache and itself (tree row 0)
    np.testing.assert_allclose(sharp[0, 0, 0], vf[int(scores.argmax()), 0], atol=1e-9)
