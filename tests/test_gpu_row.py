"""-m gpu: the fused row softmax + top-k kernel against the oracle's row step, row by row."""
import numpy as np
import pytest
import torch

import oracle
from paper_2406_17276_b200 import binding, synth
from tests import _defs
from tests._gpu import dev_table

pytestmark = pytest.mark.gpu


def _check_rows(tab, k, rows=None):
    H, V = tab.shape
    rows = np.arange(H, dtype=np.int32) if rows is None else np.asarray(rows, np.int32)
    ot = binding.OptTree(V, H, 8, k, 4, 1)
    tok, prob = ot.row_softmax_topk(dev_table(tab), torch.from_numpy(rows).cuda())
    torch.cuda.synchronize()
    assert ot.device_status() == 0
    tok, prob = tok.cpu().numpy(), prob.cpu().numpy()
    kk = min(k, V)
    worst = 0.0
    for i, r in enumerate(rows):
        etok, ep, _m, _S = oracle.row_softmax_topk(tab[r], k)
        assert tok[i, :kk].tolist() == etok.tolist(), f"row {r}"
        rel = np.abs(prob[i, :kk] - ep) / ep
        assert rel.max() <= 1e-5, f"row {r}: {rel.max():.3e}"
        worst = max(worst, float(rel.max()))
    return worst


@pytest.mark.parametrize("V,k", [(8, 2), (8, 8), (12, 5), (100, 10), (1000, 10), (4099, 32), (8192, 10), (8200, 16),
                                 (20000, 10), (32000, 10), (32000, 32), (40000, 1), (128256, 16), (152064, 32)])
def test_rows_of_synthetic_tables(V, k):
    H = 24 if V > 50000 else 64
    worst = _check_rows(_defs.small_table(H, V, 100 + V % 97), k)
    assert worst < 2e-6          # far inside the 1e-5 tolerance; guards the fp32 bulk sum


@pytest.mark.parametrize("V,k", [(640, 7), (32000, 10), (152064, 32)])
def test_constant_and_tie_heavy_rows(V, k):
    rng = np.random.default_rng(V)
    rows = [np.full(V, 1.5, np.float32),                                   # every logit ties
            np.zeros(V, np.float32),
            rng.integers(-3, 4, V).astype(np.float32),                     # 7 distinct values
            np.where(np.arange(V) % 2 == 0, 0.0, -0.0).astype(np.float32), # +0 and -0 are the same value
            np.sort(rng.standard_normal(V).astype(np.float32) * 3),        # ascending: maxima all at the end
            np.sort(rng.standard_normal(V).astype(np.float32) * 3)[::-1].copy()]
    tab = synth.f32_to_bf16_bits(np.stack(rows))
    _check_rows(tab, k)


def test_masked_vocabulary_rows():
    V, k = 32000, 10
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((4, V)) * 3).astype(np.float32)
    x[0, 100:] = -np.inf                                   # only 100 finite logits
    x[1, ::2] = -np.inf
    x[2, :] = -np.inf; x[2, 31990:] = np.arange(10, dtype=np.float32)      # exactly k finite logits at the very end
    x[3, :16000] = -np.inf
    _check_rows(synth.f32_to_bf16_bits(x), k)


def test_large_dynamic_range_rows():
    V, k = 32000, 10
    rng = np.random.default_rng(6)
    x = (rng.standard_normal((3, V)) * 3).astype(np.float32)
    x[0, 17] = 300.0                                       # one huge peak: everything else underflows
    x[1] *= 30.0                                           # very spread out
    x[2] = x[2] * 1e-3 - 200.0                             # nearly flat, far from zero
    _check_rows(synth.f32_to_bf16_bits(x), k)


def test_unaligned_table_base_takes_the_generic_path():
    V, k, H = 1000, 10, 8
    tab = _defs.small_table(H, V, 3)
    buf = torch.zeros(H * V + 1, dtype=torch.int16, device="cuda")
    buf[1:] = torch.from_numpy(tab.view(np.int16).reshape(-1)).cuda()
    view = buf[1:]                                          # base address is 2 bytes off a 16-byte boundary
    ot = binding.OptTree(V, H, 8, k, 4, 1)
    rows = torch.arange(H, dtype=torch.int32, device="cuda")
    tok, prob = ot.row_softmax_topk(view, rows)
    torch.cuda.synchronize()
    assert ot.device_status() == 0
    for r in range(H):
        etok, ep, _m, _S = oracle.row_softmax_topk(tab[r], k)
        assert tok[r].cpu().numpy().tolist() == etok.tolist()
        np.testing.assert_allclose(prob[r].cpu().numpy(), ep, rtol=1e-5)
