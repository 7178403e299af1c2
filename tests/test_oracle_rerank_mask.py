"""Pins for reranking, flattening, the ancestor mask and position ids (Section 4.2)."""
import itertools

import numpy as np
import pytest

from oracle import ref
from workloads import get_config
from workloads import generators as gen


def _tree(seed, V, k, D, B=1):
    rng = np.random.default_rng(seed)
    rows = (2.0 * rng.standard_normal((B, ref.n_draft_rows(k, D), V))).astype(np.float32)
    return ref.build_tree(rows, V, k, D)


def _level(i, k):
    return 1 if i < k else 2 + (i - k) // (k * k)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("m", [1, 5, 16, 36, 50])
def test_rerank_equals_brute_force_sort(seed, m):
    V, k, D = 200, 4, 3
    t = _tree(seed, V, k, D)
    N = ref.n_nodes(k, D)
    sel = ref.rerank(t.token, t.parent, t.value, k, D, m)
    keep = min(m, N)
    chosen = sorted(sorted(range(N), key=lambda i: (-t.value[0, i], i))[:keep])
    assert sel.n_sel[0] == keep
    assert sel.index[0, :keep].tolist() == chosen
    flat = {c: j for j, c in enumerate(chosen)}
    for j, c in enumerate(chosen):
        p = t.parent[0, c]
        assert sel.parent[0, j] == (-1 if p < 0 else flat[p])  # closure: parent is selected
        assert sel.token[0, j] == t.token[0, c]
        assert sel.depth[0, j] == _level(c, k) - 1
    assert (sel.index[0, keep:] == -1).all() and (sel.parent[0, keep:] == -1).all()
    assert sel.status == 0


def test_equal_values_prefer_shallower_node():
    # a chain whose children have probability exactly 1 relative to the parent (value equal)
    k, D, m = 2, 3, 3
    N = ref.n_nodes(k, D)
    token = np.arange(N, dtype=np.int32)[None]
    parent = np.array([[-1, -1, 0, 0, 1, 1, 2, 2, 3, 3]], np.int32)
    value = np.full((1, N), -5.0)
    value[0, [0, 2, 6]] = -1.0  # node 0, its child 2, grandchild 6 all tie
    sel = ref.rerank(token, parent, value, k, D, m)
    assert sel.index[0].tolist() == [0, 2, 6]
    sel2 = ref.rerank(token, parent, value, k, D, 2)
    assert sel2.index[0].tolist() == [0, 2]  # the shallower of the tied nodes


def test_clamp_forces_ancestors_in_for_arbitrary_values():
    k, D, m = 2, 3, 3
    N = ref.n_nodes(k, D)
    token = np.zeros((1, N), np.int32)
    parent = np.array([[-1, -1, 0, 0, 1, 1, 2, 2, 3, 3]], np.int32)
    value = np.full((1, N), -9.0)
    value[0, 6] = -0.1  # a deep node that (illegally) beats its ancestors 2 and 0
    value[0, 1] = -1.0
    sel = ref.rerank(token, parent, value, k, D, m)
    chosen = sel.index[0].tolist()
    assert sel.status == 0
    for j, c in enumerate(chosen):  # closed under parents
        assert parent[0, c] < 0 or parent[0, c] in chosen


@pytest.mark.parametrize("seed", range(5))
@pytest.mark.parametrize("m", [3, 5, 7])
def test_selection_maximises_total_value_over_connected_subsets(seed, m):
    """Exhaustive check on N = 14: no root-connected subset of size m has a larger sum of values
    (sum of path products = expected accepted length under the paper's approximation)."""
    V, k, D = 30, 2, 4
    t = _tree(40 + seed, V, k, D)
    N = ref.n_nodes(k, D)
    assert N == 14
    sel = ref.rerank(t.token, t.parent, t.value, k, D, m)
    w = np.exp(t.value[0])
    got = w[sel.index[0, :m]].sum()
    best = 0.0
    for sub in itertools.combinations(range(N), m):
        s = set(sub)
        if all(t.parent[0, i] < 0 or t.parent[0, i] in s for i in sub):
            best = max(best, w[list(sub)].sum())
    assert abs(got - best) <= 1e-15 * max(1.0, best)


def _ancestors(parent_flat, i):
    out = {i}
    a = parent_flat[i]
    while a >= 0:
        out.add(a)
        a = parent_flat[a]
    return out


@pytest.mark.parametrize("name,m", [("tiny", 16), ("tiny", 70)])
def test_mask_is_ancestor_set_and_lower_triangular(name, m):
    cfg = get_config(name)
    rows = gen.draft_rows(cfg, seed=11)
    t = ref.build_tree(rows, cfg.V, cfg.k, cfg.D)
    sel = ref.rerank(t.token, t.parent, t.value, cfg.k, cfg.D, m)
    kv_len = np.array([77], np.int32)
    bits, dense, pos, st = ref.tree_mask(sel.parent, sel.depth, sel.n_sel, kv_len, m, dense=True)
    assert st == 0
    W = (m + 63) // 64
    assert bits.shape == (1, m, W)
    ns = int(sel.n_sel[0])
    for i in range(m):
        want = _ancestors(sel.parent[0], i) if i < ns else {i}
        got = {j for j in range(m) if (int(bits[0, i, j // 64]) >> (j % 64)) & 1}
        assert got == want
        assert all(j <= i for j in got)  # lower triangular in flat (topological) order
        assert dense[0, i].nonzero()[0].tolist() == sorted(want)
        if i < ns:
            assert len(got) == sel.depth[0, i] + 1  # popcount = depth + 1
            assert pos[0, i] == 77 + sel.depth[0, i]
            p = sel.parent[0, i]
            if p >= 0:  # row i = row(parent) | bit i
                want_row = bits[0, p].copy()
                want_row[i // 64] |= np.uint64(1 << (i % 64))
                assert (bits[0, i] == want_row).all()


def test_chain_tree_gives_causal_mask():
    V, k, D, m = 50, 1, 6, 6
    t = _tree(3, V, k, D)
    sel = ref.rerank(t.token, t.parent, t.value, k, D, m)
    assert sel.parent[0].tolist() == [-1, 0, 1, 2, 3, 4]
    _, dense, pos, _ = ref.tree_mask(sel.parent, sel.depth, sel.n_sel, np.array([10], np.int32), m,
                                     dense=True)
    assert (dense[0] == np.tril(np.ones((m, m), np.uint8))).all()
    assert pos[0].tolist() == [10, 11, 12, 13, 14, 15]


def test_bad_parent_sets_status():
    sel_parent = np.array([[-1, 0, 5, 1]], np.int32)  # parent after child
    sel_depth = np.array([[0, 1, 2, 2]], np.int32)
    _, _, _, st = ref.tree_mask(sel_parent, sel_depth, np.array([4], np.int32),
                                np.array([0], np.int32), 4)
    assert st & ref.ST_BAD_TREE


@pytest.mark.parametrize("by_confidence", [False, True])
@pytest.mark.parametrize("m", [3, 12, 20, 50])
def test_without_reranking_the_draft_is_the_frontiers_of_all_steps(m, by_confidence):
    """Section 5.2, the ablation without reranking.  The frontier after every step is recorded while the
    tree is grown one step at a time (those frontiers are themselves pinned against a brute force); the
    selection must be their union, lowest indices first when it exceeds m, flattened like any other."""
    V, k, D = 60, 4, 5
    for seed in range(5):
        rng = np.random.default_rng(500 + seed)
        rows = (2.0 * rng.standard_normal((1, ref.n_draft_rows(k, D), V))).astype(np.float32)
        tree = ref.new_tree(1, k, D)
        union = set()
        for s in range(D):
            lo = 0 if s == 0 else 1 + (s - 1) * k
            n_s = 1 if s == 0 else k
            ref.expand(tree, np.ascontiguousarray(rows[:, lo:lo + n_s]), V, k, D, s, by_confidence=by_confidence)
            union |= set(tree.frontier[0].tolist())
        assert len(union) == k * D
        want = sorted(union)[:m]
        sel = ref.rerank_skipped(tree.token, tree.parent, tree.value, tree.frontier, k, D, m)
        assert sel.status == 0
        assert sel.n_sel[0] == len(want)
        assert sel.index[0, :len(want)].tolist() == want
        assert (sel.index[0, len(want):] == -1).all()
        flat = {c: j for j, c in enumerate(want)}
        for j, c in enumerate(want):
            p = tree.parent[0, c]
            assert sel.parent[0, j] == (-1 if p < 0 else flat[p])  # connected whatever m cuts off
            assert sel.token[0, j] == tree.token[0, c]
            assert sel.depth[0, j] == _level(c, k) - 1
        if not by_confidence and m >= k * D:
            # the reranked tree of the same size is at least as good under the paper's objective
            full = ref.rerank(tree.token, tree.parent, tree.value, k, D, k * D)
            assert np.exp(tree.value[0, full.index[0, :k * D]]).sum() >= \
                np.exp(tree.value[0, want]).sum() - 1e-15


def test_without_reranking_a_bad_frontier_is_reported():
    k, D, m = 2, 3, 6
    N = ref.n_nodes(k, D)
    token = np.zeros((1, N), np.int32)
    parent = np.array([[-1, -1, 0, 0, 1, 1, 2, 2, 3, 3]], np.int32)
    value = np.zeros((1, N))
    sel = ref.rerank_skipped(token, parent, value, np.array([[6, 99]], np.int32), k, D, m)
    assert sel.status & ref.ST_BAD_TREE
    assert sel.index[0, :int(sel.n_sel[0])].tolist() == [0, 1, 2, 3, 6]
