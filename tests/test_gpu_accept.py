"""GPU parity: acceptance (greedy and multi-round sampling) and KV compaction against the CPU oracle.

Accepted lengths, paths and extra tokens must be bit-exact.  A trial is exempt only where the oracle
reports that rounding could flip a decision: an acceptance test with |u - a| < 1e-6, or the extra
token's uniform within 1e-5 (relative) of a CDF boundary."""
import numpy as np
import pytest
import torch
from scipy import stats

import paper_2406_16858_b200 as e2
from oracle import ref
from workloads import get_config
from workloads import generators as gen

from harness import DEV, dev, gpu_accept, host, new_status

pytestmark = pytest.mark.gpu


# Exemptions are counted over the whole module and held to ceilings by the module's last test.
COUNTS = {"trials": 0, "decision_exempt": 0, "sampled": 0, "token_exempt": 0}


def _pipeline(cfg, seed):
    draft = gen.draft_rows(cfg, seed)
    tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    sel = ref.rerank(tree.token, tree.parent, tree.value, cfg.k, cfg.D, cfg.m)
    target = gen.target_rows(cfg, seed, draft, tree.parent, sel.index)
    ua, ub = gen.uniforms(cfg, seed)
    return draft, sel, target, ua, ub


def _compare(cfg, draft, sel, target, ua, ub, temperature, point_mass=False, t_stride=None,
             d_stride=None):
    d_arg = None if (temperature == 0 or point_mass) else draft
    want = ref.accept(target, d_arg, sel, cfg.V, cfg.k, cfg.D, cfg.m, temperature, ua, ub,
                      t_stride=t_stride, d_stride=d_stride, debug=temperature > 0)
    alen, apath, bonus, st = gpu_accept(target, d_arg, sel.index, sel.parent, sel.token, sel.n_sel,
                                        cfg.V, cfg.k, cfg.D, cfg.m, temperature, ua, ub,
                                        t_stride=t_stride, d_stride=d_stride)
    assert st == want.status
    n_exempt = 0
    for b in range(len(alen)):
        COUNTS["trials"] += 1
        COUNTS["sampled"] += temperature > 0
        if temperature > 0 and want.margins[b, 0] < 1e-6:
            n_exempt += 1
            COUNTS["decision_exempt"] += 1
            continue
        assert alen[b] == want.acc_len[b], (b, alen[b], want.acc_len[b])
        assert (apath[b] == want.acc_path[b]).all()
        if temperature > 0 and want.margins[b, 1] < 1e-5:
            # the draw falls within 1e-5 of a step of the distribution function (always so when the
            # drawn token itself holds less than 2e-5): the device may name a neighbour, but only one
            # whose own step lies within that distance of the draw
            n_exempt += 1
            COUNTS["token_exempt"] += 1
            p = want.p_final[b]
            cdf = np.cumsum(p)
            thr = float(ub[b]) * cdf[-1]
            t = int(bonus[b])
            assert 0 <= t < cfg.V and p[t] > 0
            assert cdf[t] - p[t] - 1e-5 * cdf[-1] <= thr <= cdf[t] + 1e-5 * cdf[-1], (b, t, want.bonus_token[b])
            continue
        assert bonus[b] == want.bonus_token[b], (b, bonus[b], want.bonus_token[b], want.margins[b])
    return n_exempt, want


@pytest.mark.parametrize("seed", range(100))
@pytest.mark.parametrize("temperature", [0.0, 1.0])
def test_tiny_100_seeds(seed, temperature):
    cfg = get_config("tiny")
    draft, sel, target, ua, ub = _pipeline(cfg, seed)
    _compare(cfg, draft, sel, target, ua, ub, temperature)


@pytest.mark.parametrize("seed", range(20))
def test_tiny_point_mass_and_other_temperatures(seed):
    cfg = get_config("tiny")
    draft, sel, target, ua, ub = _pipeline(cfg, seed)
    _compare(cfg, draft, sel, target, ua, ub, 1.0, point_mass=True)
    _compare(cfg, draft, sel, target, ua, ub, 0.6)
    _compare(cfg, draft, sel, target, ua, ub, 1.7)


@pytest.mark.parametrize("name,temperature", [("vicuna7b", 0.0), ("vicuna7b", 1.0), ("llama3_8b", 1.0),
                                              ("llama3_8b", 0.0)])
@pytest.mark.parametrize("seed", range(5))
def test_model_shaped(name, temperature, seed):
    cfg = get_config(name)
    draft, sel, target, ua, ub = _pipeline(cfg, seed)
    _compare(cfg, draft, sel, target, ua, ub, temperature)


@pytest.mark.parametrize("V,k,D,m,B", [(1001, 3, 4, 20, 3), (4099, 2, 5, 9, 2), (517, 8, 2, 40, 2),
                                       (70001, 4, 3, 128, 2), (250003, 3, 2, 8, 1)])
@pytest.mark.parametrize("temperature", [0.0, 1.0])
def test_odd_shapes(V, k, D, m, B, temperature):
    cfg = get_config("tiny", B=B, V=V, k=k, D=D, m=m)
    draft, sel, target, ua, ub = _pipeline(cfg, 7)
    _compare(cfg, draft, sel, target, ua, ub, temperature)
    if temperature > 0:
        _compare(cfg, draft, sel, target, ua, ub, temperature, point_mass=True)


def test_always_reject_and_always_accept_uniforms():
    cfg = get_config("tiny")
    draft, sel, target, ua, ub = _pipeline(cfg, 3)
    almost_one = np.nextafter(np.float32(1), np.float32(0))
    for u in (np.zeros_like(ua), np.full_like(ua, almost_one)):
        for bonus_u in (np.zeros_like(ub), np.full_like(ub, almost_one)):
            _compare(cfg, draft, sel, target, u, bonus_u, 1.0)


def test_target_equal_to_draft_accepts_first_children():
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
    ua, ub = gen.uniforms(cfg, 5)
    # p == q: thresholds are 1 up to rounding, so use uniforms clear of 1
    _compare(cfg, draft, sel, target, np.minimum(ua, np.float32(0.99)), ub, 1.0)


@pytest.mark.parametrize("mode", ["full_q", "point_mass"])
def test_chi_square_on_gpu_1e6_trials(mode):
    """The lossless property on the GPU path itself: 10^6 seeded trials at V = 1000, one
    verification level, siblings drawn without replacement from q (full-q rule) or the top-k children
    (point-mass rule); the first emitted token follows the target distribution."""
    cfg = get_config("tiny")
    n, c, V = 1_000_000, cfg.k, cfg.V
    draft = gen.draft_rows(cfg, seed=123)[:, :1]
    rng = np.random.default_rng(99)
    target = (draft[0, 0] + 0.5 * rng.standard_normal((c + 1, V)).astype(np.float32))[None]
    z = target[0, 0].astype(np.float64)
    p = np.exp(z - z.max())
    p /= p.sum()
    zq = draft[0, 0].astype(np.float64)
    q = np.exp(zq - zq.max())
    q /= q.sum()
    if mode == "full_q":
        cdf = np.cumsum(q) / q.sum()
        tokens = np.empty((n, c), np.int64)
        for j in range(c):
            draw = np.searchsorted(cdf, rng.random(n), side="right")
            while True:
                dup = (tokens[:, :j] == draw[:, None]).any(axis=1)
                if not dup.any():
                    break
                draw[dup] = np.searchsorted(cdf, rng.random(int(dup.sum())), side="right")
            tokens[:, j] = np.minimum(draw, V - 1)
        tokens = tokens.astype(np.int32)
        d_arg = np.ascontiguousarray(draft)
    else:
        tokens = np.tile(np.argsort(-draft[0, 0], kind="stable")[:c].astype(np.int32), (n, 1))
        d_arg = None
    sel_index = np.tile(np.arange(c, dtype=np.int32), (n, 1))
    sel_parent = np.full((n, c), -1, np.int32)
    n_sel = np.full(n, c, np.int32)
    ua = rng.random((n, c), dtype=np.float32)
    ub = rng.random(n, dtype=np.float32)
    alen, apath, bonus, st = gpu_accept(target, d_arg, sel_index, sel_parent, tokens, n_sel, V, c, 1, c,
                                        1.0, ua, ub, t_stride=0, d_stride=0)
    assert st == 0
    first = np.where(alen > 0, tokens[np.arange(n), np.maximum(apath[:, 0], 0)], bonus)
    expected = n * p
    small = expected < 10
    obs = np.bincount(first, minlength=V).astype(np.float64)
    o = np.append(obs[~small], obs[small].sum())
    e = np.append(expected[~small], expected[small].sum())
    chi2 = ((o - e) ** 2 / e).sum()
    assert stats.chi2.sf(chi2, len(e) - 1) > 1e-3


def test_kv_compact_matches_oracle_gather():
    rng = np.random.default_rng(0)
    m, D, Hkv, d, n_layers = 16, 6, 4, 64, 5
    kv_len = np.array([50, 0, 333, 7], np.int32)
    off = gen.kv_offsets(kv_len, m)
    rows = int(off[-1] + kv_len[-1] + m)
    K = [rng.integers(0, 65536, (rows, Hkv, d)).astype(np.uint16) for _ in range(n_layers)]
    Vv = [rng.integers(0, 65536, (rows, Hkv, d)).astype(np.uint16) for _ in range(n_layers)]
    acc_path = np.array([[0, 2, 3, 7, 9, 15], [1, 4, -1, -1, -1, -1], [-1] * 6, [0, 1, 2, -1, -1, -1]],
                        np.int32)
    acc_len = np.array([6, 2, 0, 3], np.int32)
    tK, tV = [dev(a) for a in K], [dev(a) for a in Vv]
    kp = torch.tensor([t.data_ptr() for t in tK], dtype=torch.int64, device=DEV)
    vp = torch.tensor([t.data_ptr() for t in tV], dtype=torch.int64, device=DEV)
    t_len = dev(kv_len.copy())
    st = new_status()
    e2.kv_compact(kp, vp, n_layers, dev(off), t_len, dev(acc_path), dev(acc_len), 4, m, D, Hkv, d, st)
    torch.cuda.synchronize()
    want_len = kv_len.copy()
    assert ref.kv_compact(K, Vv, off, want_len, acc_path, acc_len, m, D) == 0
    assert int(st.item()) == 0
    assert (host(t_len) == want_len).all()
    for layer in range(n_layers):
        for got, want in ((tK[layer], K[layer]), (tV[layer], Vv[layer])):
            g = host(got, np.uint16)
            for b in range(4):
                n_valid = int(want_len[b])
                assert (g[off[b]:off[b] + n_valid] == want[off[b]:off[b] + n_valid]).all()


def test_kv_compact_rejects_a_non_increasing_path():
    m, D, Hkv, d = 8, 3, 1, 64
    kv_len = np.array([4], np.int32)
    rows = 4 + m
    K = dev(np.arange(rows * Hkv * d, dtype=np.uint16).reshape(rows, Hkv, d))
    kp = torch.tensor([K.data_ptr()], dtype=torch.int64, device=DEV)
    t_len = dev(kv_len.copy())
    st = new_status()
    before = K.clone()
    e2.kv_compact(kp, kp, 1, dev(np.zeros(1, np.int64)), t_len, dev(np.array([[3, 2, 5]], np.int32)),
                  dev(np.array([3], np.int32)), 1, m, D, Hkv, d, st)
    torch.cuda.synchronize()
    assert int(st.item()) & e2.STATUS_BAD_TREE
    assert host(t_len)[0] == 4 and torch.equal(K, before)


def test_zz_exemptions_stay_within_their_ceilings():
    """Runs after the tests above (file order).  A decision is exempt when a uniform lies within
    1e-6 of its threshold: about one in 10^5 trials, none on this module's seeded inputs.  The extra
    token is exempt (and then checked for validity instead of identity) when its draw lies within
    1e-5 of a step of the distribution function, which is always so for a token that holds less
    than 2e-5: a few per cent of the draws at V = 1000, up to about a third at V = 32000, more at
    V = 128256."""
    assert COUNTS["decision_exempt"] <= 1 + COUNTS["trials"] // 1000, COUNTS
    assert COUNTS["token_exempt"] <= 2 + COUNTS["sampled"] // 4, COUNTS
