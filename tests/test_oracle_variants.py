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
