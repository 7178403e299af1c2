"""The paper's ablation variants (Section 5.2) on a calibrated synthetic workload, oracle only.

With targets whose greedy token is drawn from the draft distribution itself, a child is accepted with
exactly its confidence, so the expected number of accepted draft tokens of a verified tree is the sum
of the values (path products) of its nodes: the quantity the reranking maximises (Section 4.2).  That
pins expansion, selection and greedy acceptance together against a closed form, and fixes the direction
of the ablation table: the full method is at least as good as either ablation, each at least as good
as both together."""
import numpy as np
import pytest

from oracle import ref
from workloads import get_config
from workloads import generators as gen

VARIANTS = {"full": (False, False), "without_value": (True, False), "without_reranking": (False, True),
            "without_both": (True, True)}


def _run(cfg, seed, by_confidence, skip_rerank):
    draft = gen.draft_rows(cfg, seed)
    tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D, by_confidence=by_confidence)
    if skip_rerank:
        sel = ref.rerank_skipped(tree.token, tree.parent, tree.value, tree.frontier, cfg.k, cfg.D, cfg.m)
    else:
        sel = ref.rerank(tree.token, tree.parent, tree.value, cfg.k, cfg.D, cfg.m)
    target = gen.target_rows_calibrated(cfg, seed, draft, tree.parent, sel.index)
    ua, ub = gen.uniforms(cfg, seed)
    res = ref.accept(target, None, sel, cfg.V, cfg.k, cfg.D, cfg.m, 0.0, ua, ub)
    expected = np.array([np.exp(tree.value[b, sel.index[b, :int(sel.n_sel[b])]]).sum() for b in range(cfg.B)])
    return res.acc_len.astype(np.float64), expected


def test_accepted_length_matches_the_sum_of_values_and_the_ablations_order():
    cfg = get_config("tiny", B=8, k=4, D=5, m=20)  # m = kD: every variant verifies 20 tokens
    seeds = range(120)
    measured, expected = {}, {}
    for name, (by_confidence, skip) in VARIANTS.items():
        got = [_run(cfg, seed, by_confidence, skip) for seed in seeds]
        measured[name] = np.concatenate([g[0] for g in got])
        expected[name] = np.concatenate([g[1] for g in got])
    n = len(measured["full"])
    for name in VARIANTS:
        # mean of n accepted lengths against its expectation: the lengths lie in [0, D], their
        # standard deviation is below 1.2 here, so 4 standard errors is 4*1.2/sqrt(n)
        assert abs(measured[name].mean() - expected[name].mean()) < 4 * 1.2 / np.sqrt(n), name
    # per tree, exactly: reranking picks the best connected subtree of the same size
    assert (expected["full"] >= expected["without_reranking"] - 1e-12).all()
    assert (expected["without_value"] >= expected["without_both"] - 1e-12).all()
    # on average: expanding on value grows the better tree
    assert expected["full"].mean() > expected["without_value"].mean()
    assert expected["without_reranking"].mean() > expected["without_both"].mean()
    # and the measured lengths follow the same order as the paper's ablation table
    assert measured["full"].mean() > measured["without_reranking"].mean() > measured["without_both"].mean()
    assert measured["full"].mean() > measured["without_value"].mean() > measured["without_both"].mean()


def test_calibrated_targets_accept_a_child_with_its_confidence():
    """The generator's own claim, checked by counting: over many draws the greedy token of a calibrated
    row falls on a given token with that token's softmax probability."""
    cfg = get_config("tiny", B=1, V=12, k=2, D=2, m=4)
    draft = gen.draft_rows(cfg, 0)
    p = np.exp(draft[0, 0].astype(np.float64) - draft[0, 0].max())
    p /= p.sum()
    counts = np.zeros(cfg.V)
    trials = 4000
    tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    sel = ref.rerank(tree.token, tree.parent, tree.value, cfg.k, cfg.D, cfg.m)
    for seed in range(trials):
        rows = gen.target_rows_calibrated(cfg, seed, draft, tree.parent, sel.index)
        counts[int(np.argmax(rows[0, 0]))] += 1
    keep = p * trials >= 5
    chi2 = ((counts[keep] - p[keep] * trials) ** 2 / (p[keep] * trials)).sum()
    assert chi2 < 45  # 99.99th percentile of chi-square with at most 11 degrees of freedom is below 40


def test_dynamic_tree_accepts_more_than_the_fixed_shape_tree_of_the_same_size():
    """The paper's central comparison (Section 3 against Section 4) on the calibrated workload: with the
    same number of verified tokens and the same depth limit, the context-dependent tree has the larger
    expected accepted length, and both measured means sit on their expectations."""
    from scipy.special import logsumexp
    from workloads import static_tree

    k, D = 10, static_tree.N_LEVELS
    index, parent, depth, rank, row_of = static_tree.shape(k)
    n = len(index)
    cfg = get_config("tiny", B=8, V=1000, k=k, D=D, m=n)
    got = {"static": [], "dynamic": []}
    want = {"static": [], "dynamic": []}
    for seed in range(40):
        draft = gen.draft_rows(cfg, seed)
        ua, ub = gen.uniforms(cfg, seed)
        # dynamic: the method itself
        tree = ref.build_tree(draft, cfg.V, k, D)
        sel = ref.rerank(tree.token, tree.parent, tree.value, k, D, n)
        target = gen.target_rows_calibrated(cfg, seed, draft, tree.parent, sel.index)
        got["dynamic"].append(ref.accept(target, None, sel, cfg.V, k, D, n, 0.0, ua, ub).acc_len)
        want["dynamic"].append(np.exp(np.take_along_axis(tree.value, sel.index.astype(np.int64), axis=1)).sum(axis=1))
        # static: the declared shape filled with per-position top tokens
        tok = static_tree.tokens(draft, k)
        ssel = ref.Selection(np.tile(index, (cfg.B, 1)), np.tile(parent, (cfg.B, 1)), tok,
                             np.tile(depth, (cfg.B, 1)), np.full(cfg.B, n, np.int32))
        parent_cand = np.full((cfg.B, cfg.N), -1, np.int32)  # which candidate expanded which slot
        for x in range(n):
            if parent[x] >= 0:
                parent_cand[:, index[x]] = index[parent[x]]
        starget = gen.target_rows_calibrated(cfg, seed, draft, parent_cand, ssel.index)
        got["static"].append(ref.accept(starget, None, ssel, cfg.V, k, D, n, 0.0, ua, ub).acc_len)
        expect = np.zeros(cfg.B)
        for b in range(cfg.B):
            logv = np.zeros(n)
            for x in range(n):  # ascending index: parents first
                row = 0 if parent[x] < 0 else int(row_of[parent[x]])
                z = draft[b, row].astype(np.float64)
                logv[x] = (0.0 if parent[x] < 0 else logv[parent[x]]) + z[tok[b, x]] - logsumexp(z)
            expect[b] = np.exp(logv).sum()
        want["static"].append(expect)
    for name in got:
        g, w = np.concatenate(got[name]).astype(np.float64), np.concatenate(want[name])
        assert abs(g.mean() - w.mean()) < 4 * 1.2 / np.sqrt(len(g)), name
        got[name], want[name] = g, w
    assert want["dynamic"].mean() > want["static"].mean()
    assert got["dynamic"].mean() > got["static"].mean()
