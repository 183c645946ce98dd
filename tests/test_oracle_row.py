"""Pins for the oracle's row step (softmax normaliser + k most probable tokens)."""
import numpy as np
import pytest

import oracle
from paper_2406_17276_b200 import synth
from tests import _defs


@pytest.mark.parametrize("V,k,seed", [(8, 2, 1), (8, 8, 2), (1000, 10, 3), (4099, 32, 4), (32000, 10, 5)])
def test_row_matches_numpy_softmax_and_lexsort(V, k, seed):
    tab = _defs.small_table(4, V, seed)
    for r in range(tab.shape[0]):
        tok, p, m, S = oracle.row_softmax_topk(tab[r], k)
        x = synth.bf16_bits_to_f32(tab[r]).astype(np.float64)
        e = np.exp(x - x.max())
        probs = e / e.sum()
        want = _defs.np_topk(x, min(k, V))
        assert tok.tolist() == want.tolist()
        np.testing.assert_allclose(p, probs[want], rtol=1e-12)
        assert m == x.max()
        np.testing.assert_allclose(S, e.sum(), rtol=1e-12)


def test_probabilities_of_a_full_row_sum_to_one():
    tab = _defs.small_table(2, 257, 9)
    tok, p, _m, _S = oracle.row_softmax_topk(tab[1], 257)
    assert sorted(tok.tolist()) == list(range(257))
    assert abs(p.sum() - 1.0) < 1e-12


def test_constant_row_closed_form():
    V, k = 640, 7
    row = synth.f32_to_bf16_bits(np.full(V, 1.5, np.float32))
    tok, p, m, S = oracle.row_softmax_topk(row, k)
    assert tok.tolist() == list(range(k))          # ties go to the lowest token ids
    np.testing.assert_allclose(p, np.full(k, 1.0 / V), rtol=1e-13)
    assert m == 1.5 and abs(S - V) < 1e-9


def test_one_hot_biased_row_closed_form():
    V, k, c, b = 512, 3, 77, 6.0
    x = np.zeros(V, np.float32); x[c] = b
    tok, p, _m, _S = oracle.row_softmax_topk(synth.f32_to_bf16_bits(x), k)
    z = np.exp(b) + (V - 1)
    assert tok.tolist() == [c, 0, 1]
    np.testing.assert_allclose(p, [np.exp(b) / z, 1 / z, 1 / z], rtol=1e-13)


def test_ties_inside_topk_break_by_token_id():
    x = np.array([1.0, 3.0, 2.0, 3.0, 2.0, 0.0, 3.0, 2.0], np.float32)
    tok, _p, _m, _S = oracle.row_softmax_topk(synth.f32_to_bf16_bits(x), 5)
    assert tok.tolist() == [1, 3, 6, 2, 4]


def test_argmax_lowest_token_on_ties():
    x = np.array([0.5, 4.0, 4.0, -1.0], np.float32)
    assert oracle.row_argmax(synth.f32_to_bf16_bits(x)) == 1
