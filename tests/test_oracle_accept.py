"""Pins for the oracle's acceptance step: brute force for greedy, exact integration of the output
law for the multi-round sampling rule (Sections 2.1, 2.2), the textbook chain rule, closed forms,
and a chi-square test over 10^6 seeded trials at the tiny vocabulary."""
import itertools

import numpy as np
import pytest
from scipy import stats

from oracle import ref
from workloads import get_config
from workloads import generators as gen

ALMOST_ONE = np.float32(np.nextafter(np.float32(1.0), np.float32(0.0)))


def _softmax(z, t=1.0):
    z = z.astype(np.float64) / t
    e = np.exp(z - z.max())
    return e / e.sum()


def _pipeline(cfg, seed):
    draft = gen.draft_rows(cfg, seed)
    tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    sel = ref.rerank(tree.token, tree.parent, tree.value, cfg.k, cfg.D, cfg.m)
    target = gen.target_rows(cfg, seed, draft, tree.parent, sel.index)
    ua, ub = gen.uniforms(cfg, seed)
    return draft, tree, sel, target, ua, ub


# ---------------------------------------------------------------- greedy

@pytest.mark.parametrize("seed", range(20))
def test_greedy_is_longest_argmax_path(seed):
    cfg = get_config("tiny")
    draft, tree, sel, target, _, _ = _pipeline(cfg, seed)
    got = ref.accept(target, None, sel, cfg.V, cfg.k, cfg.D, cfg.m, 0.0)
    ns = int(sel.n_sel[0])
    am = target[0].argmax(axis=1)  # numpy argmax returns the lowest index on ties
    # brute force: every selected node whose whole root path matches the target argmax chain
    ok = {}
    for x in range(ns):
        p = sel.parent[0, x]
        row_of_parent = 0 if p < 0 else 1 + p
        ok[x] = (p < 0 or ok[p]) and sel.token[0, x] == am[row_of_parent]
    good = [x for x in range(ns) if ok[x]]
    depth_best = max([sel.depth[0, x] + 1 for x in good], default=0)
    assert got.acc_len[0] == depth_best
    path = got.acc_path[0, :depth_best].tolist()
    for j, x in enumerate(path):
        assert ok[x] and sel.depth[0, x] == j and sel.parent[0, x] == (path[j - 1] if j else -1)
    assert (got.acc_path[0, depth_best:] == -1).all()
    last_row = 0 if depth_best == 0 else 1 + path[-1]
    assert got.bonus_token[0] == am[last_row]


def test_greedy_accepts_a_fully_matching_chain():
    V, k, D, m = 30, 1, 4, 4
    rng = np.random.default_rng(0)
    draft = rng.standard_normal((1, ref.n_draft_rows(k, D), V)).astype(np.float32)
    tree = ref.build_tree(draft, V, k, D)
    sel = ref.rerank(tree.token, tree.parent, tree.value, k, D, m)
    target = np.zeros((1, m + 1, V), np.float32)
    for r in range(m):  # row r is the row of the parent of flat node r in a chain
        target[0, r, sel.token[0, r]] = 3.0
    target[0, m, 17] = 3.0
    got = ref.accept(target, None, sel, V, k, D, m, 0.0)
    assert got.acc_len[0] == 4 and got.acc_path[0].tolist() == [0, 1, 2, 3]
    assert got.bonus_token[0] == 17


# ---------------------------------------------------------------- temperature > 0

def _root_only_selection(tokens, B=1):
    """Selection whose nodes are all children of the root (one verification level)."""
    tokens = np.atleast_2d(np.asarray(tokens, np.int32))
    B, c = tokens.shape
    return ref.Selection(np.tile(np.arange(c, dtype=np.int32), (B, 1)), np.full((B, c), -1, np.int32),
                         np.ascontiguousarray(tokens), np.zeros((B, c), np.int32),
                         np.full(B, c, np.int32))


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("V,c", [(4, 2), (6, 3), (5, 1)])
@pytest.mark.parametrize("temperature", [1.0, 0.7])
def test_first_token_law_is_exactly_the_target_full_q(seed, V, c, temperature):
    """Integrate over every sibling draw (sequentially, without replacement from q) and every
    accept/reject outcome: the first emitted token follows p exactly."""
    rng = np.random.default_rng(1000 + seed)
    draft = (1.5 * rng.standard_normal((1, 1, V))).astype(np.float32)
    target = (1.5 * rng.standard_normal((1, c + 1, V))).astype(np.float32)
    p, q = _softmax(target[0, 0], temperature), _softmax(draft[0, 0], temperature)
    law = np.zeros(V)
    total_mass = 0.0
    for cand in itertools.permutations(range(V), c):
        pr, rest = 1.0, 1.0
        for x in cand:
            pr *= q[x] / rest
            rest -= q[x]
        sel = _root_only_selection(cand)
        u = np.full((1, c), ALMOST_ONE, np.float32)  # rejects everything: all children are tested
        out = ref.accept(target, draft, sel, V, k=c, D=1, m=c, temperature=temperature,
                         u_accept=u, u_bonus=np.zeros(1, np.float32), debug=True)
        a = out.accept_prob[0]
        reach = pr
        for j, x in enumerate(cand):
            if np.isnan(a[j]):  # accepted with certainty earlier: unreachable
                reach = 0.0
                break
            law[x] += reach * a[j]
            reach *= 1.0 - a[j]
        if reach > 0:
            assert out.acc_len[0] == 0
            law += reach * out.p_final[0] / out.p_final[0].sum()
        total_mass += pr
    assert abs(total_mass - 1.0) < 1e-12
    np.testing.assert_allclose(law, p, rtol=0, atol=1e-12)


@pytest.mark.parametrize("seed", range(6))
def test_first_token_law_point_mass_mode_with_fixed_candidates(seed):
    """draft_logits_all = None: the proposal is the point mass on each (deterministic) candidate;
    the law of the first emitted token is p for ANY fixed candidate list."""
    V, c = 7, 3
    rng = np.random.default_rng(50 + seed)
    target = (2.0 * rng.standard_normal((1, c + 1, V))).astype(np.float32)
    p = _softmax(target[0, 0])
    cand = rng.permutation(V)[:c]
    sel = _root_only_selection(cand)
    out = ref.accept(target, None, sel, V, k=c, D=1, m=c, temperature=1.0,
                     u_accept=np.full((1, c), ALMOST_ONE, np.float32),
                     u_bonus=np.zeros(1, np.float32), debug=True)
    a = out.accept_prob[0]
    law, reach, removed = np.zeros(V), 1.0, 0.0
    for j, x in enumerate(cand):
        np.testing.assert_allclose(a[j], p[x] / (1.0 - removed), rtol=1e-12)  # closed form
        law[x] += reach * a[j]
        reach *= 1.0 - a[j]
        removed += p[x]
    law += reach * out.p_final[0]
    np.testing.assert_allclose(law, p, atol=1e-12)
    want_final = p.copy()
    want_final[cand] = 0
    np.testing.assert_allclose(out.p_final[0], want_final / want_final.sum(), atol=1e-12)


def _textbook_chain(p_rows, q_rows, tokens, u_acc, u_bonus):
    """Chain speculative sampling as in Section 2.1, written directly."""
    n = len(tokens)
    for i in range(n):
        p, q = p_rows[i], q_rows[i]
        if u_acc[i] < min(1.0, p[tokens[i]] / q[tokens[i]]):
            continue
        res = np.maximum(p - q, 0.0)
        return i, int(np.searchsorted(np.cumsum(res), u_bonus * res.sum(), side="right"))
    p = p_rows[n]
    return n, int(np.searchsorted(np.cumsum(p), u_bonus * p.sum(), side="right"))


@pytest.mark.parametrize("seed", range(30))
def test_chain_tree_reduces_to_textbook_speculative_sampling(seed):
    V, k, D, m = 40, 1, 5, 5
    rng = np.random.default_rng(seed)
    draft = (1.2 * rng.standard_normal((1, ref.n_draft_rows(k, D), V))).astype(np.float32)
    tree = ref.build_tree(draft, V, k, D)
    sel = ref.rerank(tree.token, tree.parent, tree.value, k, D, m)
    target = (draft[:, :1].repeat(m + 1, axis=1) * 0).astype(np.float32)
    target[0, :m] = draft[0, :m] + 0.7 * rng.standard_normal((m, V)).astype(np.float32)
    target[0, m] = rng.standard_normal(V).astype(np.float32)
    ua = rng.random((1, m), dtype=np.float32)
    ub = rng.random(1, dtype=np.float32)
    got = ref.accept(target, draft, sel, V, k, D, m, 1.0, ua, ub)
    # chain: flat node i is at depth i; its parent's target row is row i, its draft row is row i
    p_rows = [_softmax(target[0, r]) for r in range(m + 1)]
    q_rows = [_softmax(draft[0, r]) for r in range(m)]
    n_acc, token = _textbook_chain(p_rows, q_rows, sel.token[0], ua[0].astype(np.float64), float(ub[0]))
    assert got.acc_len[0] == n_acc
    assert got.acc_path[0, :n_acc].tolist() == list(range(n_acc))
    if got.margins[0, 1] > 1e-9:
        assert got.bonus_token[0] == token


def test_identical_target_and_draft_always_accept_first_child():
    cfg = get_config("tiny")
    draft = gen.draft_rows(cfg, 5)
    tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    sel = ref.rerank(tree.token, tree.parent, tree.value, cfg.k, cfg.D, cfg.m)
    nd = gen.node_draft_rows(tree.parent, cfg.k, cfg.D)
    target = np.zeros((1, cfg.m + 1, cfg.V), np.float32)
    target[0, 0] = draft[0, 0]
    for x in range(cfg.m):
        r = nd[0, sel.index[0, x]]
        target[0, 1 + x] = draft[0, r] if r >= 0 else 0.0
    ua = np.full((1, cfg.m), ALMOST_ONE, np.float32)
    got = ref.accept(target, draft, sel, cfg.V, cfg.k, cfg.D, cfg.m, 1.0, ua, np.zeros(1, np.float32))
    # p == q at every expanded node: the first (most probable) child is accepted while one exists
    path = got.acc_path[0, :got.acc_len[0]].tolist()
    cur = -1
    for x in path:
        first_child = min(j for j in range(cfg.m) if sel.parent[0, j] == cur)
        assert x == first_child
        cur = x
    assert not any(sel.parent[0, j] == cur for j in range(int(sel.n_sel[0]))) or got.acc_len[0] == cfg.D


def test_extra_token_is_inverse_cdf_of_final_distribution():
    V = 9
    rng = np.random.default_rng(2)
    target = rng.standard_normal((1, 1 + 2, V)).astype(np.float32)
    draft = rng.standard_normal((1, 1, V)).astype(np.float32)
    sel = _root_only_selection([3, 5])
    u = np.full((1, 2), ALMOST_ONE, np.float32)
    probe = ref.accept(target, draft, sel, V, 2, 1, 2, 1.0, u, np.zeros(1, np.float32), debug=True)
    cdf = np.cumsum(probe.p_final[0])
    for t in range(V):
        lo = cdf[t - 1] if t else 0.0
        if cdf[t] - lo < 1e-6:
            continue
        mid = np.array([(lo + cdf[t]) / 2 / cdf[-1]], np.float32)
        got = ref.accept(target, draft, sel, V, 2, 1, 2, 1.0, u, mid)
        assert got.bonus_token[0] == t


def _sample_without_replacement(q, c, B, rng):
    """B sibling lists drawn sequentially from q without replacement (redraw on repeats)."""
    cdf = np.cumsum(q)
    cdf /= cdf[-1]
    out = np.empty((B, c), np.int64)
    for j in range(c):
        draw = np.searchsorted(cdf, rng.random(B), side="right")
        while True:
            dup = (out[:, :j] == draw[:, None]).any(axis=1)
            if not dup.any():
                break
            draw[dup] = np.searchsorted(cdf, rng.random(int(dup.sum())), side="right")
        out[:, j] = np.minimum(draw, len(q) - 1)
    return out.astype(np.int32)


def _chi_square_p_value(first_tokens, p, n):
    expected = n * p
    small = expected < 10
    obs = np.bincount(first_tokens, minlength=len(p)).astype(np.float64)
    o = np.append(obs[~small], obs[small].sum())
    e = np.append(expected[~small], expected[small].sum())
    keep = e > 0
    chi2 = ((o[keep] - e[keep]) ** 2 / e[keep]).sum()
    return stats.chi2.sf(chi2, keep.sum() - 1)


@pytest.mark.parametrize("mode", ["full_q", "point_mass"])
def test_chi_square_first_token_follows_target_1e6_trials(mode):
    """10^6 seeded trials at V = 1000: siblings drawn from q without replacement (full-q rule) or
    the deterministic top-k children (point-mass rule); the first emitted token must follow p."""
    cfg = get_config("tiny")
    n, c, V = 1_000_000, cfg.k, cfg.V
    draft = gen.draft_rows(cfg, seed=123)[:, :1]  # one hard/easy row as the root's draft row
    rng = np.random.default_rng(99)
    target = np.zeros((1, c + 1, V), np.float32)
    target[0] = draft[0, 0] + 0.5 * rng.standard_normal((c + 1, V)).astype(np.float32)
    p, q = _softmax(target[0, 0]), _softmax(draft[0, 0])
    if mode == "full_q":
        tokens = _sample_without_replacement(q, c, n, rng)
        d_arg = np.ascontiguousarray(draft)
    else:
        tokens = np.tile(np.argsort(-draft[0, 0], kind="stable")[:c].astype(np.int32), (n, 1))
        d_arg = None
    sel = _root_only_selection(tokens)
    ua = rng.random((n, c), dtype=np.float32)
    ub = rng.random(n, dtype=np.float32)
    out = ref.accept(target, d_arg, sel, V, k=c, D=1, m=c, temperature=1.0, u_accept=ua, u_bonus=ub,
                     t_stride=0, d_stride=0)
    first = np.where(out.acc_len > 0, tokens[np.arange(n), np.maximum(out.acc_path[:, 0], 0)],
                     out.bonus_token)
    assert _chi_square_p_value(first, p, n) > 1e-3
    # the test has teeth: the same statistic rejects the draft distribution
    assert _chi_square_p_value(first, q, n) < 1e-6


# ---------------------------------------------------------------- compaction

def test_kv_compact_is_a_gather_of_the_accepted_rows():
    rng = np.random.default_rng(0)
    m, D, Hkv, d, n_layers = 8, 4, 2, 16, 3
    kv_len = np.array([5, 0, 9], np.int32)
    off = gen.kv_offsets(kv_len, m)
    rows = int(off[-1] + kv_len[-1] + m)
    K = [rng.integers(0, 65536, (rows, Hkv, d)).astype(np.uint16) for _ in range(n_layers)]
    Vv = [rng.integers(0, 65536, (rows, Hkv, d)).astype(np.uint16) for _ in range(n_layers)]
    K0, V0 = [a.copy() for a in K], [a.copy() for a in Vv]
    acc_path = np.array([[0, 2, 3, 7], [1, 4, -1, -1], [-1, -1, -1, -1]], np.int32)
    acc_len = np.array([4, 2, 0], np.int32)
    new_len = kv_len.copy()
    assert ref.kv_compact(K, Vv, off, new_len, acc_path, acc_len, m, D) == 0
    assert new_len.tolist() == [9, 2, 9]
    for layer in range(n_layers):
        for got, orig in ((K[layer], K0[layer]), (Vv[layer], V0[layer])):
            for b in range(3):
                L = int(kv_len[b])
                assert (got[off[b]:off[b] + L] == orig[off[b]:off[b] + L]).all()  # prefix untouched
                for j in range(acc_len[b]):
                    assert (got[off[b] + L + j] == orig[off[b] + L + acc_path[b, j]]).all()
