"""GPU parity: tree-masked attention against the CPU oracle, within 2e-2 absolute (bf16 output,
fp32 accumulation), through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2406_16858_b200 as e2
from oracle import ref
from workloads import get_config
from workloads import generators as gen

from harness import DEV, dev, gpu_attention, host, make_ws, new_status

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _random_forest_mask(rng, B, m, kv_len, n_sel=None):
    parent = np.full((B, m), -1, np.int32)
    depth = np.zeros((B, m), np.int32)
    for b in range(B):
        for i in range(1, m):
            parent[b, i] = rng.integers(-1, i)
            depth[b, i] = 0 if parent[b, i] < 0 else depth[b, parent[b, i]] + 1
    ns = np.full(B, m, np.int32) if n_sel is None else n_sel
    bits, _, _, st = ref.tree_mask(parent, depth, ns, kv_len, m)
    assert st == 0
    return bits


def _inputs(seed, B, m, Hq, Hkv, d, lens):
    rng = np.random.default_rng(seed)
    kv_len = np.array(lens, np.int32)
    kv_off = gen.kv_offsets(kv_len, m)
    rows = int(kv_off[-1] + kv_len[-1] + m)
    q = gen.f32_to_bf16_bits(rng.standard_normal((B, m, Hq, d)).astype(np.float32))
    kc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
    vc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
    return q, kc, vc, kv_off, kv_len, _random_forest_mask(rng, B, m, kv_len)


def _compare(q, kc, vc, kv_off, kv_len, bits, scale, samples=None):
    got, lse, st = gpu_attention(q, kc, vc, kv_off, kv_len, bits, scale, want_lse=True)
    assert st == 0
    gf = gen.bf16_bits_to_f32(got).astype(np.float64)
    if samples is None:
        _, want, wlse = ref.tree_attention(q, kc, vc, kv_off, kv_len, bits, scale, want_lse=True)
        assert np.abs(gf - want).max() <= TOL
        assert np.abs(lse - wlse).max() <= 2e-2
    else:
        _, want, wlse = ref.tree_attention(q, kc, vc, kv_off, kv_len, bits, scale, samples=samples,
                                           want_lse=True)
        for t, (b, h, i) in enumerate(samples):
            assert np.abs(gf[b, i, h] - want[t]).max() <= TOL
            assert abs(lse[b, h, i] - wlse[t]) <= 2e-2
    return gf


@pytest.mark.parametrize("seed", range(5))
def test_tiny_config(seed):
    cfg = get_config("tiny")
    q, kc, vc, off, kl, bits = _inputs(seed, 1, cfg.m, cfg.Hq, cfg.Hkv, cfg.d, [cfg.kv_len])
    _compare(q, kc, vc, off, kl, bits, 1.0 / np.sqrt(cfg.d))


@pytest.mark.parametrize("m,Hq,Hkv,d,lens", [
    (16, 4, 4, 64, [0]),            # no cache at all: tree rows only
    (16, 4, 4, 64, [1]),
    (60, 8, 2, 128, [63]),          # GQA g=4, a single partly filled tile
    (60, 8, 2, 128, [64, 65, 4]),   # tile boundaries, ragged batch
    (60, 8, 1, 128, [300]),         # g=8: two row blocks
    (128, 4, 1, 64, [777]),         # largest m, two mask words
    (7, 2, 2, 64, [129, 1000]),
    (60, 32, 8, 128, [2050, 31]),
    (1, 1, 1, 128, [500]),
])
def test_shapes_tails_and_gqa(m, Hq, Hkv, d, lens):
    q, kc, vc, off, kl, bits = _inputs(11, len(lens), m, Hq, Hkv, d, lens)
    _compare(q, kc, vc, off, kl, bits, 1.0 / np.sqrt(d))


@pytest.mark.parametrize("m,Hq,Hkv,d,lens", [
    # query heads per KV head that do not divide 256: a row block holds whole tokens only, so the
    # blocks are sized from 256 // g tokens (g = 7: 36 tokens = 252 rows; g = 6: 42 tokens = 252 rows)
    (73, 7, 1, 128, [900]),           # three row blocks, several splits (one sequence, one KV head)
    (73, 7, 1, 128, [40] * 40),       # the same rows written directly: one split per sequence
    (128, 6, 1, 128, [1500]),         # four row blocks of 32 tokens
    (128, 6, 1, 64, [77] * 30),
    (109, 7, 1, 64, [300, 5]),
    (85, 6, 2, 128, [2000, 130]),
])
def test_row_blocks_when_the_group_size_does_not_divide_256(m, Hq, Hkv, d, lens):
    q, kc, vc, off, kl, bits = _inputs(17, len(lens), m, Hq, Hkv, d, lens)
    rng = np.random.default_rng(m)
    n = 500
    samples = np.stack([rng.integers(0, len(lens), n), rng.integers(0, Hq, n),
                        rng.integers(0, m, n)], axis=1).astype(np.int32)
    samples[:Hq] = [(0, h, m - 1) for h in range(Hq)]  # the last token's rows: the tail of the last row block
    _compare(q, kc, vc, off, kl, bits, 1.0 / np.sqrt(d), samples=samples)


@pytest.mark.parametrize("m,Hq,Hkv,d,lens", [
    # many (sequence, KV head) pairs leave one split per sequence: several tiles per block, so the
    # K/V ring and the score slots are reused; ragged lengths leave some blocks a single tile
    (60, 16, 16, 128, [700, 100, 1500, 40, 2100, 300, 900, 5]),      # one 128-row tile per block
    (60, 32, 8, 128, [2300, 64, 513, 1200, 1, 0, 777, 1800, 130, 260, 2047, 90, 400, 33, 1024, 640]),
    (33, 8, 8, 64, [1500, 257, 900, 31, 2000, 5, 640, 128, 129, 1100]),  # head_dim 64, deeper ring
])
def test_many_tiles_per_block(m, Hq, Hkv, d, lens):
    q, kc, vc, off, kl, bits = _inputs(23, len(lens), m, Hq, Hkv, d, lens)
    rng = np.random.default_rng(5)
    n = 400
    samples = np.stack([rng.integers(0, len(lens), n), rng.integers(0, Hq, n),
                        rng.integers(0, m, n)], axis=1).astype(np.int32)
    _compare(q, kc, vc, off, kl, bits, 1.0 / np.sqrt(d), samples=samples)


def test_ragged_batch_runs_longest_first_with_several_splits():
    """192 (sequence, KV head) pairs and sequences of up to 71 tiles: the launch is ordered by a
    device-built list, long sequences are cut into splits of 32 tiles and merged, short ones write
    their rows directly, two sequences are empty."""
    m, Hq, Hkv, d = 60, 32, 8, 128
    lens = [9000, 300, 4500, 20, 70, 5200, 1300, 0, 4037, 4036, 8100, 64, 2500, 1, 700, 3100,
            128, 4097, 0, 950, 6000, 33, 2047, 410]
    q, kc, vc, off, kl, bits = _inputs(31, len(lens), m, Hq, Hkv, d, lens)
    rng = np.random.default_rng(6)
    n = 600
    samples = np.stack([rng.integers(0, len(lens), n), rng.integers(0, Hq, n),
                        rng.integers(0, m, n)], axis=1).astype(np.int32)
    _compare(q, kc, vc, off, kl, bits, 1.0 / np.sqrt(d), samples=samples)


@pytest.mark.parametrize("m,Hq,Hkv,d,B,longest", [
    (33, 8, 8, 64, 20, 6000),    # head_dim 64: deeper K/V ring, two splits for the longest sequences
    (40, 6, 2, 128, 80, 5000),   # three query heads per KV head: query rows copied by hand, not by TMA
    (60, 32, 8, 128, 8, 16384),  # few long sequences on block pairs: four and five splits merged inside the kernel
    (60, 3, 1, 128, 37, 16384),  # short blocks: eight and nine splits per long sequence (nine: one row per warp at a time)
])
def test_ordered_launch_other_shapes(m, Hq, Hkv, d, B, longest):
    rng = np.random.default_rng(B + d)
    lens = rng.integers(0, 900, B)
    lens[[1, B // 2, B - 2]] = [longest, longest - 1700, longest - 300]
    # the device-built list and the attention kernel, which merges the splits itself: no merge launch
    assert e2.tree_attention_launches(B, m, Hq, Hkv, d, longest) == 2
    q, kc, vc, off, kl, bits = _inputs(41, B, m, Hq, Hkv, d, [int(x) for x in lens])
    n = 500
    samples = np.stack([rng.integers(0, B, n), rng.integers(0, Hq, n), rng.integers(0, m, n)], axis=1).astype(np.int32)
    samples[:60, 0] = np.array([1, B // 2, B - 2])[rng.integers(0, 3, 60)]  # the split sequences for sure
    _compare(q, kc, vc, off, kl, bits, 1.0 / np.sqrt(d), samples=samples)


def test_draft_side_attention_over_the_growing_tree():
    """The draft model's own attention while it expands the tree (Section 4.1): at step s the k
    frontier tokens attend to the committed cache and to their ancestors among the tokens expanded
    so far.  The tokens fed so far - k per step, in feeding order - are the tree rows of the call, so
    the same entry point serves it at m = s*k; the tree is the one the oracle's expansion builds."""
    V, k, D, B = 500, 10, 6, 2
    Hq, Hkv, d = 32, 8, 128
    rng = np.random.default_rng(12)
    draft = (2.0 * rng.standard_normal((B, ref.n_draft_rows(k, D), V))).astype(np.float32)
    tree = ref.new_tree(B, k, D)
    fed = [[] for _ in range(B)]  # candidate indices of the tokens fed to the draft model so far
    kv_len = np.array([700, 129], np.int32)
    for s in range(D):
        lo = 0 if s == 0 else 1 + (s - 1) * k
        ref.expand(tree, draft.reshape(-1)[lo * V:], V, k, D, s, batch_stride=draft.shape[1] * V)
        if s == D - 1:
            break  # the last level is never fed back
        for b in range(B):
            fed[b] += [int(x) for x in tree.frontier[b]]
        m = (s + 1) * k
        parent = np.full((B, m), -1, np.int32)
        depth = np.zeros((B, m), np.int32)
        for b in range(B):
            where = {c: i for i, c in enumerate(fed[b])}
            for i, c in enumerate(fed[b]):
                pc = int(tree.parent[b, c])
                if pc >= 0:  # an ancestor of a frontier token was itself a frontier token earlier
                    parent[b, i] = where[pc]
                    depth[b, i] = depth[b, where[pc]] + 1
        bits, _, _, st = ref.tree_mask(parent, depth, np.full(B, m, np.int32), kv_len, m)
        assert st == 0
        kv_off = gen.kv_offsets(kv_len, m)
        rows = int(kv_off[-1] + kv_len[-1] + m)
        q = gen.f32_to_bf16_bits(rng.standard_normal((B, m, Hq, d)).astype(np.float32))
        kc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
        vc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
        new = np.arange(m - k, m)  # the step's own queries: every head of the k newest tokens
        samples = np.array([(b, h, i) for b in range(B) for h in (0, 5, Hq - 1) for i in new], np.int32)
        _compare(q, kc, vc, kv_off, kv_len, bits, 1.0 / np.sqrt(d), samples=samples)


def test_rows_after_a_sequence_may_hold_anything():
    """The kernel streams whole tiles, so it reads cache rows that follow a sequence's last key; their
    contents (here NaN and Inf bit patterns) must not reach the output."""
    m, Hq, Hkv, d = 16, 4, 2, 64
    kv_len = np.array([70, 3], np.int32)
    kv_off = np.array([0, 200], np.int64)  # slack between and after the sequences
    rows = 400
    rng = np.random.default_rng(2)
    q = gen.f32_to_bf16_bits(rng.standard_normal((2, m, Hq, d)).astype(np.float32))
    kc = np.full((rows, Hkv, d), 0x7FC0, np.uint16)  # NaN
    vc = np.full((rows, Hkv, d), 0x7F80, np.uint16)  # +Inf
    for b in range(2):
        lo, hi = int(kv_off[b]), int(kv_off[b] + kv_len[b] + m)
        kc[lo:hi] = gen.f32_to_bf16_bits(rng.standard_normal((hi - lo, Hkv, d)).astype(np.float32))
        vc[lo:hi] = gen.f32_to_bf16_bits(rng.standard_normal((hi - lo, Hkv, d)).astype(np.float32))
    bits = _random_forest_mask(rng, 2, m, kv_len)
    _compare(q, kc, vc, kv_off, kv_len, bits, 0.125)


def test_sequence_outside_the_cache_is_reported_and_skipped():
    m, Hq, Hkv, d = 16, 2, 2, 64
    q, kc, vc, off, kl, bits = _inputs(3, 2, m, Hq, Hkv, d, [50, 60])
    tq, tk, tv = dev(q), dev(kc), dev(vc)
    out = torch.full((2, m, Hq, d), 0x1234, dtype=torch.int16, device=DEV)
    st = new_status()
    ws = make_ws(e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=2, m=m, Hq=Hq, Hkv=Hkv, d=d, max_kv_len=60))
    bad_len = np.array([50, 61], np.int32)  # sequence 1 claims more rows than max_kv_len allows
    e2.tree_attention(tq, tk, tv, kc.shape[0], dev(off), dev(bad_len), dev(bits), 2, m, Hq, Hkv, d, 60,
                      0.125, out, None, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == e2.STATUS_KV_OVERFLOW
    got = host(out, np.uint16)
    assert (got[1] == 0x1234).all()  # untouched
    _, want, _ = ref.tree_attention(q, kc, vc, off, kl, bits, 0.125)
    assert np.abs(gen.bf16_bits_to_f32(got[0]).astype(np.float64) - want[0]).max() <= TOL


def test_padding_rows_see_only_themselves_and_cache():
    rng = np.random.default_rng(0)
    m, H, d, L = 16, 2, 64, 40
    q, kc, vc, off, kl, _ = _inputs(5, 1, m, H, H, d, [L])
    bits = _random_forest_mask(rng, 1, m, kl, n_sel=np.array([9], np.int32))
    _compare(q, kc, vc, off, kl, bits, 0.125)


def test_large_scores_do_not_overflow():
    q, kc, vc, off, kl, bits = _inputs(6, 1, 16, 2, 2, 64, [200])
    _compare(q, kc, vc, off, kl, bits, 3.0)  # sharply peaked softmax


@pytest.mark.parametrize("name", ["vicuna7b", "llama3_8b", "llama2_70b"])
def test_full_size_one_layer_sampled(name):
    """Full model-shaped sizes, the launch configuration the benchmark times; the oracle computes sampled
    (sequence, head, query) rows one by one."""
    cfg = get_config(name)
    g = torch.Generator(device=DEV).manual_seed(1234)
    kv_len = gen.kv_lengths(cfg, 0)
    kv_off = gen.kv_offsets(kv_len, cfg.m)
    rows = int(kv_off[-1] + kv_len[-1] + cfg.m)
    tq = torch.randn((cfg.B, cfg.m, cfg.Hq, cfg.d), generator=g, device=DEV).to(torch.bfloat16)
    tk = torch.randn((rows, cfg.Hkv, cfg.d), generator=g, device=DEV).to(torch.bfloat16)
    tv = torch.randn((rows, cfg.Hkv, cfg.d), generator=g, device=DEV).to(torch.bfloat16)
    draft = gen.draft_rows(cfg, 0)
    tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    sel = ref.rerank(tree.token, tree.parent, tree.value, cfg.k, cfg.D, cfg.m)
    bits, _, _, _ = ref.tree_mask(sel.parent, sel.depth, sel.n_sel, kv_len, cfg.m)
    out = torch.zeros_like(tq)
    st = new_status()
    ws = make_ws(e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=cfg.B, m=cfg.m, Hq=cfg.Hq, Hkv=cfg.Hkv,
                                    d=cfg.d, max_kv_len=int(kv_len.max())))
    e2.tree_attention(tq, tk, tv, rows, dev(kv_off), dev(kv_len), dev(bits), cfg.B, cfg.m, cfg.Hq, cfg.Hkv,
                      cfg.d, int(kv_len.max()), 1.0 / np.sqrt(cfg.d), out, None, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    rng = np.random.default_rng(1)
    n = 48
    samples = np.stack([rng.integers(0, cfg.B, n), rng.integers(0, cfg.Hq, n),
                        rng.integers(0, cfg.m, n)], axis=1).astype(np.int32)
    samples[0] = (0, 0, 0)
    samples[1] = (cfg.B - 1, cfg.Hq - 1, cfg.m - 1)
    _, want, _ = ref.tree_attention(host(tq.view(torch.int16), np.uint16), host(tk.view(torch.int16), np.uint16),
                                    host(tv.view(torch.int16), np.uint16), kv_off, kv_len, bits,
                                    1.0 / np.sqrt(cfg.d), samples=samples)
    got = out.float().cpu().numpy().astype(np.float64)
    for t, (b, h, i) in enumerate(samples):
        err = np.abs(got[b, i, h] - want[t]).max()
        assert err <= TOL
        # Design budget.  With thousands of N(0,1) keys the outputs have rms ~0.02-0.03: the bar above
        # alone could not see a wrong tree mask here (removing every ancestor moves these outputs by
        # ~3e-3).  Probabilities rounded to bf16 (2^-9 relative, random sign) and one bf16 rounding of
        # the row give ~3e-3 * |o| ~ 1e-4; 1e-3 leaves a margin of ten and is a third of a mask's worth.
        assert err <= 1e-3
    # property that holds at any size: rows are finite and bounded by the largest |v|
    assert torch.isfinite(out.float()).all()
    assert out.float().abs().max() <= tv.float().abs().max()


@pytest.mark.parametrize("mode,B,Hq,Hkv,lens", [
    ("block pairs, several splits", 1, 32, 8, [4096]),
    ("block pairs, two row blocks", 1, 64, 8, [8192]),
    ("one row tile per block", 1, 32, 32, [1024]),
    ("two row tiles per block", 8, 32, 8, [2000] * 8),
    ("ordered launch, splits merged in the kernel", 24, 32, 8,
     [9000, 300, 4500, 20, 70, 5200, 1300, 0, 4037, 4036, 8100, 64, 2500, 1, 700, 3100, 128, 4097, 0, 950, 6000,
      33, 2047, 410]),
])
def test_full_size_tree_keys_dominate(mode, B, Hq, Hkv, lens):
    """Full-size launches of every mode in which the tree tokens' keys and all queries share one
    direction (a score offset of sqrt(d) = 11.3 for every tree key), so that the tree keys a row may
    see carry most of its softmax weight: an ancestor mask applied wrongly (a bit dropped, a sibling
    let in, a row's word shifted) then moves the output by O(1), far above the bar.  The tree is a
    random forest; the oracle computes sampled rows one by one."""
    m, d = 60, 128
    rng = np.random.default_rng(len(mode))
    kv_len = np.array(lens, np.int32)
    kv_off = gen.kv_offsets(kv_len, m)
    rows = int(kv_off[-1] + kv_len[-1] + m)
    g = torch.Generator(device=DEV).manual_seed(77)
    w = torch.randn(d, generator=g, device=DEV)
    w = w / w.norm() * float(np.sqrt(d))
    tq = (torch.randn((B, m, Hq, d), generator=g, device=DEV) + w).to(torch.bfloat16)
    tk = torch.randn((rows, Hkv, d), generator=g, device=DEV)
    for b in range(B):
        lo = int(kv_off[b] + kv_len[b])
        tk[lo:lo + m] += w  # tree keys: q.k / sqrt(d) gains |w|^2 / sqrt(d) = sqrt(d)
    tk = tk.to(torch.bfloat16)
    tv = torch.randn((rows, Hkv, d), generator=g, device=DEV).to(torch.bfloat16)
    bits = _random_forest_mask(rng, B, m, kv_len)
    out = torch.zeros_like(tq)
    st = new_status()
    max_len = int(kv_len.max())
    ws = make_ws(e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=B, m=m, Hq=Hq, Hkv=Hkv, d=d, max_kv_len=max_len))
    e2.tree_attention(tq, tk, tv, rows, dev(kv_off), dev(kv_len), dev(bits), B, m, Hq, Hkv, d, max_len,
                      1.0 / np.sqrt(d), out, None, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    n = 160
    samples = np.stack([rng.integers(0, B, n), rng.integers(0, Hq, n), rng.integers(0, m, n)], axis=1).astype(np.int32)
    samples[:8, 2] = m - 1  # deep rows: the most ancestors
    samples[8:16, 0] = int(np.argmax(kv_len))
    hq, hk, hv = (host(t.view(torch.int16), np.uint16) for t in (tq, tk, tv))
    _, want, _ = ref.tree_attention(hq, hk, hv, kv_off, kv_len, bits, 1.0 / np.sqrt(d), samples=samples)
    # the same rows with every ancestor hidden (each row sees itself and the cache): how far a wrong mask moves them
    self_only = np.zeros_like(bits)
    for i in range(m):
        self_only[:, i, i // 64] = np.uint64(1) << np.uint64(i % 64)
    _, blind, _ = ref.tree_attention(hq, hk, hv, kv_off, kv_len, self_only, 1.0 / np.sqrt(d), samples=samples)
    has_anc = np.array([bin(int(bits[b, i, 0])).count("1") > 1 for b, _, i in samples])
    assert np.median(np.abs(want - blind).max(axis=1)[has_anc]) > 0.3  # the case does what it is for
    got = out.float().cpu().numpy().astype(np.float64)
    for t, (b, h, i) in enumerate(samples):
        # outputs reach |o| ~ 3 here, where bf16 steps are 2^-6: the bar scales with rows above 1
        assert np.abs(got[b, i, h] - want[t]).max() <= TOL * max(1.0, np.abs(want[t]).max())
