"""The give-up path of the kernels that wait on the device, exercised without breaking anything.

The tensor-path kernels and the streaming expansion hand tiles and candidates between warps through
barriers and queues, and every such wait is bounded.  ``eagle2_set_wait_limit`` makes that bound a
launch-time value; with a bound of a few dozen cycles the first wait of an otherwise normal call
that is not satisfied at once (the first tile has not arrived from memory yet) runs out.  The call
must then raise ``EAGLE2_STATUS_TIMEOUT``, end normally with everything it holds given back (its
outputs are undefined), and the next call with the default bound, on the same buffers and the same
workspace, must be correct: tensor memory freed, arrival counters at zero, no copy still writing
into shared memory that now belongs to another block.  Nothing here faults, traps or spins without
a bound."""
import numpy as np
import pytest
import torch

import paper_2406_16858_b200 as e2
from oracle import ref
from workloads import generators as gen

from harness import DEV, GpuTree, dev, host, make_ws, new_status

pytestmark = pytest.mark.gpu

SHORT = 64  # cycles: far below the time the first bytes need to arrive from memory


@pytest.fixture
def short_wait():
    e2.set_wait_limit(SHORT)
    yield
    e2.set_wait_limit(0)


def test_the_limit_is_a_setting_that_can_be_read_back():
    default = e2.set_wait_limit(1000)
    assert default == 1 << 31
    assert e2.set_wait_limit(0) == 1000
    assert e2.set_wait_limit(-5) == default  # <= 0 means the default


@pytest.mark.parametrize("mode,m,Hq,Hkv,d,lens", [
    ("block pair", 60, 32, 8, 128, [700]),
    ("two row tiles", 60, 32, 8, 128, [300] * 10),
    ("one row tile, queries copied by hand", 40, 6, 2, 128, [500, 90]),
    ("head_dim 64", 16, 4, 4, 64, [900]),
    ("ordered launch", 60, 32, 8, 128, [5000] + [100] * 23),
])
def test_attention_gives_up_and_recovers(short_wait, mode, m, Hq, Hkv, d, lens):
    B = len(lens)
    rng = np.random.default_rng(len(mode))
    kv_len = np.array(lens, np.int32)
    kv_off = gen.kv_offsets(kv_len, m)
    rows = int(kv_off[-1] + kv_len[-1] + m)
    q = gen.f32_to_bf16_bits(rng.standard_normal((B, m, Hq, d)).astype(np.float32))
    kc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
    vc = gen.f32_to_bf16_bits(rng.standard_normal((rows, Hkv, d)).astype(np.float32))
    bits = np.zeros((B, m, (m + 63) // 64), np.uint64)
    for i in range(m):  # a chain
        for j in range(i + 1):
            bits[:, i, j // 64] |= np.uint64(1) << np.uint64(j % 64)
    tq, tk, tv, toff, tlen, tbits = dev(q), dev(kc), dev(vc), dev(kv_off), dev(kv_len), dev(bits)
    out = torch.zeros((B, m, Hq, d), dtype=torch.int16, device=DEV)
    max_len = int(kv_len.max())
    ws = make_ws(e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=B, m=m, Hq=Hq, Hkv=Hkv, d=d, max_kv_len=max_len))
    scale = 1.0 / np.sqrt(d)

    def call():
        st = new_status()
        e2.tree_attention(tq, tk, tv, rows, toff, tlen, tbits, B, m, Hq, Hkv, d, max_len, scale, out, None, ws, st)
        torch.cuda.synchronize()
        return int(st.item())

    assert call() & e2.STATUS_TIMEOUT
    assert call() & e2.STATUS_TIMEOUT  # and again: the first give-up left nothing behind
    e2.set_wait_limit(0)
    assert call() == 0
    _, want, _ = ref.tree_attention(q, kc, vc, kv_off, kv_len, bits, scale)
    got = gen.bf16_bits_to_f32(host(out, np.uint16)).astype(np.float64)
    assert np.abs(got - want).max() <= 2e-2


def test_lm_head_gives_up_and_recovers(short_wait):
    rows, H, V = 10, 512, 40000  # more vocabulary tiles than resident blocks: rings and accumulators are reused
    hb, wb = gen.lm_head_inputs(rows, H, V, seed=3)
    th, tw = dev(hb), dev(wb)
    out = torch.zeros((rows, V), dtype=torch.float32, device=DEV)

    def call():
        st = new_status()
        e2.lm_head(th, tw, rows, H, V, out, st)
        torch.cuda.synchronize()
        return int(st.item())

    assert call() & e2.STATUS_TIMEOUT
    assert call() & e2.STATUS_TIMEOUT
    e2.set_wait_limit(0)
    assert call() == 0
    want = ref.lm_head(hb, wb)
    S = np.abs(gen.bf16_bits_to_f32(hb)).astype(np.float64) @ np.abs(gen.bf16_bits_to_f32(wb)).astype(np.float64).T
    assert (np.abs(host(out) - want) <= (H / 16 + 16) * 2.0 ** -23 * S + 1e-30).all()


def test_fused_lm_head_gives_up_and_recovers(short_wait):
    B, k, D, H, V = 16, 10, 2, 128, 40000  # 160 rows; more vocabulary tiles than blocks
    hb, wb = gen.lm_head_inputs(B * k, H, V, seed=9)
    th, tw = dev(hb), dev(wb)
    N = k + (D - 1) * k * k
    token = torch.full((B, N), -1, dtype=torch.int32, device=DEV)
    parent = torch.full((B, N), -2, dtype=torch.int32, device=DEV)
    value = torch.full((B, N), float("-inf"), dtype=torch.float64, device=DEV)
    frontier = torch.arange(k, dtype=torch.int32, device=DEV).repeat(B, 1).contiguous()
    value[:, :k] = 0.0  # level 1 as if already built: every parent has value log 1
    ws = make_ws(e2.workspace_bytes(e2.OP_LM_HEAD_EXPAND, B=B, V=V, k=k, D=D))

    def call():
        st = new_status()
        fr = frontier.clone()
        e2.lm_head_expand(th, tw, H, B, V, k, D, 1, token, parent, value, fr, ws, st)
        torch.cuda.synchronize()
        return int(st.item()), fr

    assert call()[0] & e2.STATUS_TIMEOUT
    assert call()[0] & e2.STATUS_TIMEOUT
    e2.set_wait_limit(0)
    status, fr = call()
    assert status == 0
    # level 2 of every sequence: the k best tokens of each of its k rows (the oracle's LM head)
    want_logits = ref.lm_head(hb, wb).reshape(B, k, V)
    got = host(token)[:, k:k + k * k].reshape(B, k, k)
    for b in range(B):
        for r in range(k):
            top = -np.sort(-want_logits[b, r])[:k + 1]
            if (np.diff(-top) < 1e-4).any():
                continue
            assert (got[b, r] == np.argsort(-want_logits[b, r], kind="stable")[:k]).all()


def test_streaming_expansion_gives_up_and_recovers(short_wait):
    V, k, D, B = 70004, 5, 2, 32  # 160 rows at the second step: several tiles per block, selector warp
    rng = np.random.default_rng(8)
    draft = (2.0 * rng.standard_normal((B, ref.n_draft_rows(k, D), V))).astype(np.float32)
    t_draft = dev(draft)
    gpu = GpuTree(B, V, k, D)
    gpu.expand_all(t_draft)
    assert int(gpu.status.item()) & e2.STATUS_TIMEOUT
    e2.set_wait_limit(0)
    gpu.status.zero_()
    gpu.expand_all(t_draft)  # the same tree arrays and the same workspace
    assert int(gpu.status.item()) == 0
    want = ref.build_tree(draft, V, k, D)
    assert (host(gpu.token) == want.token).all()
    assert (host(gpu.parent) == want.parent).all()
    assert (host(gpu.frontier) == want.frontier).all()
    assert np.abs(host(gpu.value) - want.value).max() < 3e-6
