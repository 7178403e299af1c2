"""GPU parity of the LM head in front of the expansion (Section 4.1) against the CPU oracle.

Bar.  Operands are bf16, so every product is exact in fp32; the tensor path adds them into an fp32
accumulator 16 terms per instruction.  Each of the H/16 accumulations rounds (or truncates) once at
a magnitude of at most S = sum_h |x_h w_h|, so |error| <= (H/16 + 16) * 2^-23 * S; the oracle sums in
double.  The test uses that bound per output and prints nothing else; observed errors are far below."""
import numpy as np
import pytest
import torch

import paper_2406_16858_b200 as e2
from oracle import ref
from workloads import get_config
from workloads import generators as gen

from harness import DEV, GpuTree, dev, host, new_status

pytestmark = pytest.mark.gpu


def _gpu_logits(hb, wb):
    rows, H = hb.shape
    V = wb.shape[0]
    out = torch.full((rows, V), float("nan"), dtype=torch.float32, device=DEV)
    st = new_status()
    e2.lm_head(dev(hb), dev(wb), rows, H, V, out, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return host(out)


def _bound(hb, wb, H):
    S = np.abs(gen.bf16_bits_to_f32(hb)).astype(np.float64) @ np.abs(gen.bf16_bits_to_f32(wb)).astype(np.float64).T
    return (H / 16 + 16) * 2.0 ** -23 * S + 1e-30


@pytest.mark.parametrize("rows,H,V", [
    (1, 64, 1), (1, 64, 128), (4, 128, 129), (10, 320, 1000), (13, 64, 5000), (16, 128, 127),
    (17, 192, 300), (40, 64, 1000), (51, 256, 2049), (200, 128, 777), (256, 64, 1000),
    (257, 64, 300), (600, 128, 1000),  # more rows than one pass holds
])
def test_small_shapes_tails_and_row_counts(rows, H, V):
    hb, wb = gen.lm_head_inputs(rows, H, V, seed=rows + V)
    got = _gpu_logits(hb, wb)
    want = ref.lm_head(hb, wb)
    assert np.isfinite(got).all()
    assert (np.abs(got - want) <= _bound(hb, wb, H)).all()


def test_more_tiles_than_blocks_and_every_stage_reused():
    # 148 blocks walk 200 vocabulary tiles; 16 K blocks per tile cycle the ring several times
    rows, H, V = 10, 1024, 200 * 128 - 5
    hb, wb = gen.lm_head_inputs(rows, H, V, seed=5)
    got = _gpu_logits(hb, wb)
    want = ref.lm_head(hb, wb)
    assert (np.abs(got - want) <= _bound(hb, wb, H)).all()


@pytest.mark.parametrize("name,H", [("vicuna7b", 4096), ("llama3_8b", 4096), ("llama2_70b", 8192)])
def test_model_shapes_sampled_vocabulary_rows(name, H):
    """Full vocabulary and hidden size on the device; the oracle computes a sample of 3000 vocabulary
    rows (the same weight rows handed to it as a smaller matrix) plus the first and last tile."""
    cfg = get_config(name)
    rows = cfg.k
    hb, wb = gen.lm_head_inputs(rows, H, cfg.V, seed=11)
    got = _gpu_logits(hb, wb)
    rng = np.random.default_rng(2)
    pick = np.unique(np.concatenate([rng.integers(0, cfg.V, 3000), np.arange(128), np.arange(cfg.V - 128, cfg.V)]))
    want = ref.lm_head(hb, np.ascontiguousarray(wb[pick]))
    err = np.abs(got[:, pick] - want)
    assert (err <= _bound(hb, wb[pick], H)).all()
    assert err.max() < 1e-4  # typical: a few 1e-6 on logits of standard deviation 2
    assert np.isfinite(got).all()


def test_refusals():
    hb, wb = gen.lm_head_inputs(4, 64, 100, seed=1)
    out = torch.zeros((4, 100), dtype=torch.float32, device=DEV)
    st = new_status()
    th, tw = dev(hb), dev(wb)
    with pytest.raises(e2.Eagle2Error) as err:
        e2.lm_head(th, tw, 4, 48, 100, out, st)      # H not a multiple of 64
    assert err.value.code == -2
    with pytest.raises(e2.Eagle2Error) as err:
        e2.lm_head(th, tw, -1, 64, 100, out, st)
    assert err.value.code == -2
    with pytest.raises(e2.Eagle2Error) as err:
        e2.lm_head(th.data_ptr() + 2, tw, 4, 64, 100, out, st)
    assert err.value.code == -3
    e2.lm_head(th, tw, 0, 64, 100, out, st)          # nothing to do
    torch.cuda.synchronize()
    assert int(st.item()) == 0


@pytest.mark.parametrize("name,H", [("tiny", 128), ("vicuna7b", 1024)])
def test_lm_head_feeds_the_expansion(name, H):
    """Features -> logits -> tree, all on the device, against the oracle's LM head and expansion.  The
    device logits carry the fp32 accumulation error, so a row is exempt where two of the oracle's
    k+1 largest logits are closer than 1e-4 (ten times the error observed), and values are compared to 1e-3."""
    cfg = get_config(name)
    checked = 0
    for seed in range(6):
        hb, wb = gen.lm_head_inputs(cfg.R, H, cfg.V, seed=40 + seed)
        want_logits = ref.lm_head(hb, wb)
        top = -np.sort(-want_logits, axis=1)[:, :cfg.k + 1]
        if (np.diff(-top, axis=1) < 1e-4).any():
            continue
        want = ref.build_tree(want_logits.astype(np.float32)[None], cfg.V, cfg.k, cfg.D)
        near_tie = False
        for s in range(cfg.D):  # a frontier decided by less than the logits' error may flip
            base = 0 if s == 0 else cfg.k + (s - 1) * cfg.k * cfg.k
            v = -np.sort(-want.value[0, base:base + (cfg.k if s == 0 else cfg.k * cfg.k)])
            near_tie |= len(v) > cfg.k and v[cfg.k - 1] - v[cfg.k] < 1e-4
        if near_tie:
            continue
        checked += 1
        logits = torch.zeros((1, cfg.R, cfg.V), dtype=torch.float32, device=DEV)
        st = new_status()
        e2.lm_head(dev(hb), dev(wb), cfg.R, H, cfg.V, logits, st)
        gpu = GpuTree(1, cfg.V, cfg.k, cfg.D).expand_all(logits)
        assert int(st.item()) == 0 and int(gpu.status.item()) == 0
        assert (host(gpu.token) == want.token).all() and (host(gpu.parent) == want.parent).all()
        assert np.abs(host(gpu.value) - want.value).max() < 1e-3
        assert (host(gpu.frontier) == want.frontier).all()
    assert checked > 0


def test_lm_head_and_expansion_replay_from_a_captured_graph():
    """Both calls only enqueue work, so the pair can be captured once and replayed: the replay on new
    features must give the logits and the tree of the plain calls."""
    cfg = get_config("tiny")
    H = 128
    hb, wb = gen.lm_head_inputs(cfg.R, H, cfg.V, seed=60)
    hb2, _ = gen.lm_head_inputs(cfg.R, H, cfg.V, seed=61)
    th, tw = dev(hb), dev(wb)
    logits = torch.zeros((1, cfg.R, cfg.V), dtype=torch.float32, device=DEV)
    st = new_status()
    tree = GpuTree(1, cfg.V, cfg.k, cfg.D)
    stream = torch.cuda.Stream()

    def enqueue():
        e2.lm_head(th, tw, cfg.R, H, cfg.V, logits, st, stream=stream)
        for s in range(cfg.D):
            lo = 0 if s == 0 else 1 + (s - 1) * cfg.k
            e2.expand(logits.data_ptr() + lo * cfg.V * 4, cfg.R * cfg.V, 1, cfg.V, cfg.k, cfg.D, s, tree.token,
                      tree.parent, tree.value, tree.frontier, tree.ws, tree.status, stream=stream)

    with torch.cuda.stream(stream):
        enqueue()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            enqueue()
        th.copy_(dev(hb2))
        graph.replay()
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and int(tree.status.item()) == 0
    want_logits = ref.lm_head(hb2, wb)
    assert (np.abs(host(logits)[0] - want_logits) <= _bound(hb2, wb, H)).all()
    want = ref.build_tree(host(logits), cfg.V, cfg.k, cfg.D)  # the tree of exactly these fp32 logits
    assert (host(tree.token) == want.token).all() and (host(tree.parent) == want.parent).all()
    assert (host(tree.frontier) == want.frontier).all()
