"""Pins for the oracle's expansion step (Section 4.1): log-softmax and top-k against numpy/scipy,
node values against brute-force path products in linear space, frontier against a brute-force sort."""
import numpy as np
import pytest
from scipy.special import logsumexp

from oracle import ref
from workloads import get_config
from workloads import generators as gen


def _small_rows(seed, B, R, V):
    rng = np.random.default_rng(seed)
    return (2.0 * rng.standard_normal((B, R, V))).astype(np.float32)


@pytest.mark.parametrize("V,k", [(17, 3), (1000, 4), (4099, 10)])
def test_step0_logsoftmax_topk_match_numpy(V, k):
    D = 2
    rows = _small_rows(1, 3, ref.n_draft_rows(k, D), V)
    tree = ref.build_tree(rows, V, k, D)
    for b in range(3):
        z = rows[b, 0].astype(np.float64)
        logp = z - logsumexp(z)
        assert abs(np.exp(logp).sum() - 1.0) < 1e-12
        order = np.argsort(-z, kind="stable")[:k]  # stable: lower token id first on ties
        assert (tree.token[b, :k] == order).all()
        assert (tree.parent[b, :k] == -1).all()
        np.testing.assert_allclose(tree.value[b, :k], logp[order], rtol=0, atol=1e-12)


def test_topk_ties_prefer_lower_token_id():
    V, k, D = 50, 4, 1
    rows = np.zeros((1, 1, V), np.float32)
    rows[0, 0, [7, 3, 30, 41, 12]] = 5.0  # five equal maxima
    tree = ref.build_tree(rows, V, k, D)
    assert tree.token[0].tolist() == [3, 7, 12, 30]
    assert tree.frontier[0].tolist() == [0, 1, 2, 3]  # equal values -> lower candidate index


def _brute(rows, V, k, D, by_confidence=False):
    """Linear-space reconstruction: softmax probabilities multiplied along every root path; the frontier
    is ranked by that product, or by each node's own probability in the ablation."""
    prob = np.exp(rows.astype(np.float64) - rows.astype(np.float64).max(axis=1, keepdims=True))
    prob /= prob.sum(axis=1, keepdims=True)
    N = k + (D - 1) * k * k
    token, parent, edge = np.zeros(N, int), np.zeros(N, int), np.zeros(N)
    lin = np.zeros(N)
    frontier, frontiers = None, []
    for s in range(D):
        n_rows = 1 if s == 0 else k
        base = 0 if s == 0 else k + (s - 1) * k * k
        new = []
        for j in range(n_rows):
            row = 0 if s == 0 else 1 + (s - 1) * k + j
            par = -1 if s == 0 else frontier[j]
            best = sorted(range(V), key=lambda v: (-float(rows[row, v]), v))[:k]
            for c, v in enumerate(best):
                node = base + j * k + c
                token[node], parent[node], edge[node] = v, par, prob[row, v]
                new.append(node)
        for node in new:  # enumerate the path root -> node, multiply in linear space
            prod, a = 1.0, node
            while a >= 0:
                prod *= edge[a]
                a = parent[a]
            lin[node] = prod
        score = edge if by_confidence else lin
        frontier = sorted(new, key=lambda n: (-score[n], n))[:k]
        frontiers.append(frontier)
    return token, parent, lin, frontiers


@pytest.mark.parametrize("seed", range(8))
def test_values_and_frontier_match_linear_space_brute_force(seed):
    V, k, D = 40, 3, 4
    R = ref.n_draft_rows(k, D)
    rows = _small_rows(100 + seed, 1, R, V)
    tree = ref.new_tree(1, k, D)
    for s in range(D):
        lo = 0 if s == 0 else 1 + (s - 1) * k
        n_s = 1 if s == 0 else k
        ref.expand(tree, np.ascontiguousarray(rows[:, lo:lo + n_s]), V, k, D, s)
        token, parent, lin, frontiers = _brute(rows[0], V, k, D)
        assert tree.frontier[0].tolist() == frontiers[s]
    assert (tree.token[0] == token).all()
    assert (tree.parent[0] == parent).all()
    np.testing.assert_allclose(np.exp(tree.value[0]), lin, rtol=1e-12)
    # Section 4.2: a node's value never exceeds its parent's
    for i in range(len(parent)):
        if parent[i] >= 0:
            assert tree.value[0, i] <= tree.value[0, parent[i]]
    assert tree.status == 0


@pytest.mark.parametrize("seed", range(6))
def test_expanding_on_confidence_matches_brute_force(seed):
    """Section 5.2, the ablation without the value: the nodes to expand are the k best of the step by
    their own softmax probability; the stored value is still the path product.  The trees must also
    differ from the value-ranked ones somewhere, or the switch would be untested."""
    V, k, D = 40, 3, 4
    rows = _small_rows(300 + seed, 1, ref.n_draft_rows(k, D), V)
    tree = ref.new_tree(1, k, D)
    for s in range(D):
        lo = 0 if s == 0 else 1 + (s - 1) * k
        n_s = 1 if s == 0 else k
        ref.expand(tree, np.ascontiguousarray(rows[:, lo:lo + n_s]), V, k, D, s, by_confidence=True)
        token, parent, lin, frontiers = _brute(rows[0], V, k, D, by_confidence=True)
        assert tree.frontier[0].tolist() == frontiers[s]
    assert (tree.token[0] == token).all() and (tree.parent[0] == parent).all()
    np.testing.assert_allclose(np.exp(tree.value[0]), lin, rtol=1e-12)
    whole = ref.build_tree(rows, V, k, D, by_confidence=True)
    assert (whole.value[0] == tree.value[0]).all() and (whole.parent[0] == tree.parent[0]).all()
    for i in range(len(parent)):  # values are path products here too: never above the parent's
        assert parent[i] < 0 or tree.value[0, i] <= tree.value[0, parent[i]]


def test_expanding_on_confidence_changes_some_frontier():
    V, k, D = 40, 3, 4
    changed = 0
    for seed in range(6):
        rows = _small_rows(300 + seed, 1, ref.n_draft_rows(k, D), V)
        a = ref.build_tree(rows, V, k, D)
        b = ref.build_tree(rows, V, k, D, by_confidence=True)
        assert (a.value[0, :k + k * k] == b.value[0, :k + k * k]).all()  # two levels share their parents
        changed += not (a.parent[0] == b.parent[0]).all()
    assert changed > 0


def test_tiny_config_generator_tree_is_consistent():
    cfg = get_config("tiny")
    rows = gen.draft_rows(cfg, seed=3)
    tree = ref.build_tree(rows, cfg.V, cfg.k, cfg.D)
    token, parent, lin, frontiers = _brute(rows[0], cfg.V, cfg.k, cfg.D)
    assert (tree.token[0] == token).all() and (tree.parent[0] == parent).all()
    np.testing.assert_allclose(np.exp(tree.value[0]), lin, rtol=1e-12)
    assert tree.frontier[0].tolist() == frontiers[-1]


def test_nonfinite_logit_sets_status():
    V, k, D = 30, 2, 2
    rows = _small_rows(5, 1, ref.n_draft_rows(k, D), V)
    rows[0, 0, 4] = np.nan
    tree = ref.build_tree(rows, V, k, D)
    assert tree.status & ref.ST_NONFINITE_LOGIT


def test_batch_entries_are_independent():
    V, k, D = 64, 3, 3
    rows = _small_rows(9, 4, ref.n_draft_rows(k, D), V)
    whole = ref.build_tree(rows, V, k, D)
    for b in range(4):
        one = ref.build_tree(np.ascontiguousarray(rows[b:b + 1]), V, k, D)
        assert (one.token[0] == whole.token[b]).all()
        assert (one.value[0] == whole.value[b]).all()
