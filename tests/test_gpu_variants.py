"""GPU parity for the paper's variants (Section 5.2 ablation; Appendix A budgets): expansion that
ranks by confidence alone, and the per-model draft-token budgets m = 50 and m = 48.

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
    _check_tree(cfg, draft, gpu, want)


@pytest.mark.parametrize("name,B", [("vicuna7b", 1), ("llama3_8b", 1), ("llama3_8b", 5)])
@pytest.mark.parametrize("seed", range(3))
def test_model_shaped_tree_ranked_by_confidence(name, B, seed):
    cfg = get_config(name, B=B)
    draft = gen.draft_rows(cfg, 50 + seed)
    want = ref.build_tree(draft, cfg.V, cfg.k, cfg.D, by_confidence=True)
    by_value = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    assert not (want.parent == by_value.parent).all()  # the switch changes the tree on this input
    gpu = GpuTree(cfg.B, cfg.V, cfg.k, cfg.D).expand_all(dev(draft), flags=e2.EXPAND_BY_CONFIDENCE)
    _check_tree(cfg, draft, gpu, want)
    # scores are not monotone along a path here: the selection relies on the ancestor rule
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
