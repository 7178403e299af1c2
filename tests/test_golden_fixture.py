"""The stored expectation under ``tests/golden/``: the oracle still reproduces it (a tripwire for changes
in the oracle's arithmetic), its contents obey what the paper fixes (Section 4: values are path
products that never exceed the parent's, the draft is a connected tree, a token sees its ancestors only),
and the device path reproduces it without calling the oracle."""
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden"))
import make_caption_shape_cycle as fixture  # noqa: E402


def _stored():
    with open(fixture.PATH) as f:
        return fixture.parse(f.read())


def test_oracle_reproduces_the_stored_cycle():
    want, got = _stored(), fixture.compute()
    assert set(want) == set(got)
    for key in want:
        if key == "tree_value":
            assert np.array_equal(np.array(want[key]), np.array(got[key]))  # repr round-trips doubles
        else:
            assert want[key] == got[key], key


def test_stored_cycle_obeys_the_papers_structure():
    d = _stored()
    k, D, m = 2, 3, 8
    par, val = d["tree_parent"], d["tree_value"]
    assert len(par) == k + (D - 1) * k * k
    for i, p in enumerate(par):
        assert p < i and (p < 0 or val[i] <= val[p])
    order = sorted(range(len(val)), key=lambda i: (-val[i], i))[:m]
    assert sorted(order) == d["sel_index"]
    chosen = d["sel_index"]
    for j, c in enumerate(chosen):
        p = par[c]
        assert d["sel_parent"][j] == (-1 if p < 0 else chosen.index(p))
        bits, a = 0, j
        while a >= 0:
            bits |= 1 << a
            a = d["sel_parent"][a]
        assert d["mask_bits"][j] == bits
        assert d["pos_ids"][j] == 17 + d["sel_depth"][j]
    assert d["acc_path"][:d["acc_len"]] == [x for x in d["acc_path"] if x >= 0]


@pytest.mark.gpu
def test_device_path_reproduces_the_stored_cycle():
    import torch

    import paper_2406_16858_b200  # noqa: F401
    from harness import GpuSelection, GpuTree, dev, gpu_accept, host
    from workloads import generators as gen

    d = _stored()
    cfg = fixture.config()
    draft = gen.draft_rows(cfg, fixture.SEED)
    tree = GpuTree(1, cfg.V, cfg.k, cfg.D).expand_all(dev(draft))
    assert host(tree.token)[0].tolist() == d["tree_token"]
    assert host(tree.parent)[0].tolist() == d["tree_parent"]
    assert np.abs(host(tree.value)[0] - np.array(d["tree_value"])).max() < 1e-5
    assert host(tree.frontier)[0].tolist() == d["frontier"]
    sel = GpuSelection(tree.token, tree.parent, tree.value, 1, cfg.k, cfg.D, cfg.m,
                       kv_len=torch.full((1,), cfg.kv_len, dtype=torch.int32, device="cuda:0"))
    assert host(sel.index)[0].tolist() == d["sel_index"] and host(sel.parent)[0].tolist() == d["sel_parent"]
    assert host(sel.token)[0].tolist() == d["sel_token"] and host(sel.depth)[0].tolist() == d["sel_depth"]
    assert host(sel.mask_bits, np.uint64)[0, :, 0].tolist() == d["mask_bits"]
    assert host(sel.pos_ids)[0].tolist() == d["pos_ids"]
    target = gen.target_rows(cfg, fixture.SEED, draft, np.array([d["tree_parent"]], np.int32),
                             np.array([d["sel_index"]], np.int32))
    ua, ub = gen.uniforms(cfg, fixture.SEED)
    alen, apath, bonus, st = gpu_accept(target, None, host(sel.index), host(sel.parent), host(sel.token),
                                        host(sel.n_sel), cfg.V, cfg.k, cfg.D, cfg.m, 0.0, ua, ub)
    assert st == d["status"] == 0
    assert int(alen[0]) == d["acc_len"] and apath[0].tolist() == d["acc_path"] and int(bonus[0]) == d["bonus_token"]
