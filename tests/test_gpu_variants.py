"""GPU parity for the paper's variants (Section 5.2 ablations; Appendix A budgets): expansion that picks
the nodes to expand by confidence instead of value, the selection without reranking, and the per-model
draft-token budgets m = 50 and m = 48.

Bar as for the default path: tokens, parents, frontier and selections bit-exact, stored scores within
1e-5 relative (3e-6 absolute on the logarithm)."""
import numpy as np
import pytest
import torch

import paper_2406_16858_b200 as e2
from oracle import ref
from workloads import get_config
from workloads import generators as gen

from harness import GpuSelection, GpuTree, dev, host
from test_gpu_tree import _check_selection, _check_tree

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(30))
def test_tiny_tree_ranked_by_confidence(seed):
    cfg = get_config("tiny")
    draft = gen.draft_rows(cfg, seed)
    want = ref.build_tree(draft, cfg.V, cfg.k, cfg.D, by_confidence=True)
    gpu = GpuTree(cfg.B, cfg.V, cfg.k, cfg.D).expand_all(dev(draft), flags=e2.EXPAND_BY_CONFIDENCE)
    _check_tree(cfg, draft, gpu, want, by_confidence=True)


@pytest.mark.parametrize("name,B", [("vicuna7b", 1), ("llama3_8b", 1), ("llama3_8b", 5)])
@pytest.mark.parametrize("seed", range(3))
def test_model_shaped_tree_ranked_by_confidence(name, B, seed):
    cfg = get_config(name, B=B)
    draft = gen.draft_rows(cfg, 50 + seed)
    want = ref.build_tree(draft, cfg.V, cfg.k, cfg.D, by_confidence=True)
    by_value = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    assert not (want.parent == by_value.parent).all()  # the switch changes the tree on this input
    gpu = GpuTree(cfg.B, cfg.V, cfg.k, cfg.D).expand_all(dev(draft), flags=e2.EXPAND_BY_CONFIDENCE)
    _check_tree(cfg, draft, gpu, want, by_confidence=True)
    _check_selection(want, cfg.k, cfg.D, cfg.m, kv_len=np.full(cfg.B, cfg.kv_len, np.int32))


def test_variant_with_no_flag_is_the_default_and_unknown_flags_are_refused():
    cfg = get_config("vicuna7b")
    draft = dev(gen.draft_rows(cfg, 7))
    a = GpuTree(cfg.B, cfg.V, cfg.k, cfg.D).expand_all(draft)
    b = GpuTree(cfg.B, cfg.V, cfg.k, cfg.D)
    R = cfg.R
    for s in range(cfg.D):
        lo = 0 if s == 0 else 1 + (s - 1) * cfg.k
        e2.expand_variant(draft.data_ptr() + lo * cfg.V * 4, R * cfg.V, cfg.B, cfg.V, cfg.k, cfg.D, s, 0,
                          b.token, b.parent, b.value, b.frontier, b.ws, b.status)
    torch.cuda.synchronize()
    assert torch.equal(a.token, b.token) and torch.equal(a.parent, b.parent)
    assert torch.equal(a.value, b.value) and torch.equal(a.frontier, b.frontier)
    with pytest.raises(e2.Eagle2Error) as err:
        e2.expand_variant(draft, R * cfg.V, cfg.B, cfg.V, cfg.k, cfg.D, 0, 2, b.token, b.parent, b.value,
                          b.frontier, b.ws, b.status)
    assert err.value.code == -2


@pytest.mark.parametrize("name,m", [("llama2_70b", 48), ("vicuna7b", 50), ("llama3_8b", 48)])
@pytest.mark.parametrize("by_confidence", [False, True])
def test_per_model_budgets_select_and_mask(name, m, by_confidence):
    """Appendix A: 50 draft tokens for the 13B models (7B-shaped vocabulary) and 48 for the 70B ones."""
    cfg = get_config(name, m=m)
    for seed in range(3):
        draft = gen.draft_rows(cfg, 20 + seed)
        want = ref.build_tree(draft, cfg.V, cfg.k, cfg.D, by_confidence=by_confidence)
        _check_selection(want, cfg.k, cfg.D, m, kv_len=np.full(cfg.B, cfg.kv_len, np.int32))


@pytest.mark.parametrize("name,m,lens", [("llama2_70b", 48, [700]), ("vicuna7b", 50, [333, 64])])
def test_per_model_budgets_attention(name, m, lens):
    import test_gpu_attention as ta
    cfg = get_config(name, m=m)
    q, kc, vc, off, kl, bits = ta._inputs(3, len(lens), m, cfg.Hq // 4, max(1, cfg.Hkv // 4), cfg.d, lens)
    ta._compare(q, kc, vc, off, kl, bits, 1.0 / np.sqrt(cfg.d))


@pytest.mark.parametrize("name,m", [("llama2_70b", 48), ("vicuna7b", 50)])
@pytest.mark.parametrize("temperature", [0.0, 1.0])
def test_per_model_budgets_acceptance(name, m, temperature):
    import test_gpu_accept as tc
    cfg = get_config(name, m=m)
    for seed in range(3):
        draft, sel, target, ua, ub = tc._pipeline(cfg, 30 + seed)
        tc._compare(cfg, draft, sel, target, ua, ub, temperature)


def _gpu_selection_without_reranking(tree: ref.Tree, k, D, m):
    B = tree.token.shape[0]
    z = lambda *shape: torch.full(shape, 77, dtype=torch.int32, device="cuda:0")  # noqa: E731
    out = [z(B, m), z(B, m), z(B, m), z(B, m), z(B)]
    st = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    e2.rerank_skipped(dev(tree.token), dev(tree.parent), dev(tree.value), dev(tree.frontier), B, k, D, m,
                      *out, st)
    torch.cuda.synchronize()
    return [host(t) for t in out], int(st.item())


@pytest.mark.parametrize("name,B,m", [("tiny", 1, 16), ("tiny", 3, 5), ("vicuna7b", 1, 60), ("llama3_8b", 2, 60),
                                      ("llama2_70b", 1, 48), ("vicuna7b", 1, 128)])
@pytest.mark.parametrize("by_confidence", [False, True])
def test_selection_without_reranking(name, B, m, by_confidence):
    """Section 5.2 ablations "without reranking" and "without both": the expansion phase's own selection,
    bit-exact against the oracle, then through the mask kernel."""
    cfg = get_config(name, B=B, m=m)
    for seed in range(3):
        draft = gen.draft_rows(cfg, 70 + seed)
        tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D, by_confidence=by_confidence)
        want = ref.rerank_skipped(tree.token, tree.parent, tree.value, tree.frontier, cfg.k, cfg.D, m)
        (idx, par, tok, dep, ns), st = _gpu_selection_without_reranking(tree, cfg.k, cfg.D, m)
        assert st == want.status == 0
        assert (ns == want.n_sel).all() and (ns == min(m, cfg.k * cfg.D)).all()
        assert (idx == want.index).all() and (par == want.parent).all()
        assert (tok == want.token).all() and (dep == want.depth).all()
        kv_len = np.full(B, cfg.kv_len, np.int32)
        wbits, _, wpos, wst = ref.tree_mask(want.parent, want.depth, want.n_sel, kv_len, m)
        W = (m + 63) // 64
        bits = torch.zeros((B, m, W), dtype=torch.int64, device="cuda:0")
        pos = torch.zeros((B, m), dtype=torch.int32, device="cuda:0")
        st2 = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        e2.tree_mask(dev(par), dev(dep), dev(ns), dev(kv_len), B, m, bits, None, pos, st2)
        torch.cuda.synchronize()
        assert int(st2.item()) == wst == 0
        assert (host(bits, np.uint64) == wbits).all() and (host(pos) == wpos).all()


def test_selection_without_reranking_from_the_gpu_tree_and_a_bad_frontier():
    """End to end on the device: the frontier the expansion kernel left feeds the selection directly.
    A frontier entry outside the tree is reported and skipped, as in the oracle."""
    cfg = get_config("vicuna7b")
    draft = gen.draft_rows(cfg, 5)
    want_tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    want = ref.rerank_skipped(want_tree.token, want_tree.parent, want_tree.value, want_tree.frontier,
                              cfg.k, cfg.D, cfg.m)
    gpu = GpuTree(cfg.B, cfg.V, cfg.k, cfg.D).expand_all(dev(draft))
    z = lambda *shape: torch.zeros(shape, dtype=torch.int32, device="cuda:0")  # noqa: E731
    out = [z(1, cfg.m), z(1, cfg.m), z(1, cfg.m), z(1, cfg.m), z(1)]
    st = z(1)
    e2.rerank_skipped(gpu.token, gpu.parent, gpu.value, gpu.frontier, 1, cfg.k, cfg.D, cfg.m, *out, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert (host(out[0]) == want.index).all() and (host(out[1]) == want.parent).all()

    bad = want_tree.frontier.copy()
    bad[0, 3] = cfg.N + 5
    want_bad = ref.rerank_skipped(want_tree.token, want_tree.parent, want_tree.value, bad, cfg.k, cfg.D, cfg.m)
    st.zero_()
    e2.rerank_skipped(gpu.token, gpu.parent, gpu.value, dev(bad), 1, cfg.k, cfg.D, cfg.m, *out, st)
    torch.cuda.synchronize()
    assert int(st.item()) == want_bad.status == e2.STATUS_BAD_TREE
    assert (host(out[4]) == want_bad.n_sel).all() and (host(out[0]) == want_bad.index).all()
    with pytest.raises(e2.Eagle2Error):
        e2.rerank_skipped(gpu.token, gpu.parent, gpu.value, None, 1, cfg.k, cfg.D, cfg.m, *out, st)


@pytest.mark.parametrize("variant", ["full", "without_value", "without_reranking", "without_both"])
@pytest.mark.parametrize("name,kw", [("tiny", dict(B=8, k=4, D=5, m=20)), ("vicuna7b", dict(B=2))])
def test_ablation_pipelines_end_to_end_on_the_device(variant, name, kw):
    """Expansion, selection, mask and greedy acceptance of each ablation variant, run on the device from
    the draft logits on, against the oracle's pipeline on calibrated targets (a child is accepted with
    its confidence): same trees, same selections, same accepted paths."""
    from harness import gpu_accept
    by_confidence = variant in ("without_value", "without_both")
    skip = variant in ("without_reranking", "without_both")
    cfg = get_config(name, **kw)
    for seed in range(4 if name == "tiny" else 2):
        draft = gen.draft_rows(cfg, 90 + seed)
        tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D, by_confidence=by_confidence)
        if skip:
            want = ref.rerank_skipped(tree.token, tree.parent, tree.value, tree.frontier, cfg.k, cfg.D, cfg.m)
        else:
            want = ref.rerank(tree.token, tree.parent, tree.value, cfg.k, cfg.D, cfg.m)
        gpu = GpuTree(cfg.B, cfg.V, cfg.k, cfg.D).expand_all(
            dev(draft), flags=e2.EXPAND_BY_CONFIDENCE if by_confidence else 0)
        _check_tree(cfg, draft, gpu, tree, by_confidence=by_confidence)
        z = lambda *shape: torch.zeros(shape, dtype=torch.int32, device="cuda:0")  # noqa: E731
        idx, par, tok, dep, ns = z(cfg.B, cfg.m), z(cfg.B, cfg.m), z(cfg.B, cfg.m), z(cfg.B, cfg.m), z(cfg.B)
        st = z(1)
        if skip:
            e2.rerank_skipped(gpu.token, gpu.parent, gpu.value, gpu.frontier, cfg.B, cfg.k, cfg.D, cfg.m,
                              idx, par, tok, dep, ns, st)
        else:
            e2.rerank(gpu.token, gpu.parent, gpu.value, cfg.B, cfg.k, cfg.D, cfg.m, idx, par, tok, dep, ns, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        if not (host(idx) == want.index).all():
            # only a near-tie in the reranked values may move a selection
            v = np.sort(tree.value, axis=1)[:, ::-1]
            assert not skip and (v[:, cfg.m - 1] - v[:, cfg.m] < 1e-6).any()
            continue
        assert (host(par) == want.parent).all() and (host(tok) == want.token).all()
        target = gen.target_rows_calibrated(cfg, 90 + seed, draft, tree.parent, want.index)
        ua, ub = gen.uniforms(cfg, 90 + seed)
        res = ref.accept(target, None, want, cfg.V, cfg.k, cfg.D, cfg.m, 0.0, ua, ub)
        alen, apath, bonus, ast = gpu_accept(target, None, host(idx), host(par), host(tok), host(ns),
                                             cfg.V, cfg.k, cfg.D, cfg.m, 0.0, ua, ub)
        assert ast == res.status
        assert (alen == res.acc_len).all() and (apath == res.acc_path).all()
        assert (bonus == res.bonus_token).all()
