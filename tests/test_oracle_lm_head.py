"""Pins for the oracle's LM head (Section 4.1: the draft feature goes through the original LLM's LM
head to give the draft distribution): a library matrix product and closed forms."""
import numpy as np
import pytest

from oracle import ref
from workloads import generators as gen


@pytest.mark.parametrize("rows,H,V", [(1, 8, 5), (10, 64, 300), (7, 130, 1001)])
def test_matches_numpy_matmul(rows, H, V):
    rng = np.random.default_rng(rows * 1000 + V)
    hb = gen.f32_to_bf16_bits(rng.standard_normal((rows, H)).astype(np.float32))
    wb = gen.f32_to_bf16_bits(rng.standard_normal((V, H)).astype(np.float32))
    got = ref.lm_head(hb, wb)
    want = gen.bf16_bits_to_f32(hb).astype(np.float64) @ gen.bf16_bits_to_f32(wb).astype(np.float64).T
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12 * H)


def test_one_hot_feature_selects_a_weight_column_and_operands_are_not_transposed():
    H, V = 16, 9
    rng = np.random.default_rng(3)
    w = rng.standard_normal((V, H)).astype(np.float32)
    wb = gen.f32_to_bf16_bits(w)
    hidden = np.zeros((2, H), np.float32)
    hidden[0, 5] = 1.0
    hidden[1, 11] = -2.0
    got = ref.lm_head(gen.f32_to_bf16_bits(hidden), wb)
    wf = gen.bf16_bits_to_f32(wb).astype(np.float64)
    assert (got[0] == wf[:, 5]).all()
    assert (got[1] == -2.0 * wf[:, 11]).all()


def test_exact_where_fp32_would_round():
    # 2^12 + 2^-12 needs 25 bits: exact in double, lost by a float accumulator
    H = 2
    hb = gen.f32_to_bf16_bits(np.array([[2.0 ** 6, 2.0 ** -6]], np.float32))
    wb = gen.f32_to_bf16_bits(np.array([[2.0 ** 6, 2.0 ** -6]], np.float32))
    assert ref.lm_head(hb, wb)[0, 0] == 2.0 ** 12 + 2.0 ** -12
