"""-m gpu: the layer-by-layer build (logits handed in per layer) gives the oracle's trees, and
opt_tree_build's bit for bit.

The table model plays the draft model: the test gathers, for every node to expand, its row of the
draft table (row of token t at depth d, as everywhere) into a dense buffer and hands that in.
"""
import math

import numpy as np
import pytest
import torch

from paper_2406_17276_b200 import binding, synth
from tests import _compare
from tests._gpu import dev_table, poison, poisoned_tree, record_parity, tree_dict

pytestmark = pytest.mark.gpu
NEG_INF = -math.inf
FIELDS = ("token", "parent", "depth", "phat", "n_sel", "depth_reached", "expected_len", "esub_trace")


def _run(w, delta, H=None, V=None, test_id=None):
    ld, lt = synth.make_tables(w, H=H, V=V)
    Hh, Vv = ld.shape
    ot = binding.OptTree(Vv, Hh, w.n, w.k, w.max_depth, w.batch)
    d_ld = dev_table(ld)                                              # [H][V] int16 view
    roots = synth.root_tokens(w.batch, Vv, w.seed + 6)
    r = torch.from_numpy(roots).cuda()
    want = ot.build(d_ld, r, delta)
    tree = poisoned_tree(ot, w.batch)
    ot.layers_begin(w.batch)
    toks = r.view(-1, 1).to(torch.int64)                              # the root is the one node to expand first
    cnt = torch.ones(w.batch, dtype=torch.int32, device="cuda")
    layers = 0
    for depth in range(0, w.max_depth + 1):
        stride = max(1, int(cnt.max().item()))
        if int(cnt.max().item()) == 0:
            break
        rows = (toks[:, :stride] * 31 + depth) % Hh                   # [B][stride]; rows beyond a count are arbitrary but valid
        rows = rows.clamp_(0, Hh - 1)
        logits = d_ld[rows.reshape(-1)].reshape(w.batch, stride, Vv).contiguous()
        nt, npar, cnt = ot.layers_step(logits, delta, tree)
        toks = nt.to(torch.int64)
        layers += 1
    torch.cuda.synchronize()
    assert ot.device_status() == 0
    assert int(cnt.max().item()) == 0, "every tree must have stopped by the depth limit"
    # against the oracle (the mask is computed from the layer-by-layer trees as well)
    g = tree_dict(tree)
    mask, pos = poison(torch.empty((w.batch, w.n, ot.W), dtype=torch.int64, device="cuda"),
                       torch.empty((w.batch, w.n), dtype=torch.int32, device="cuda"))
    ot.mask(tree, None, mask, pos)
    g.update(mask=mask.cpu().numpy(), position_ids=pos.cpu().numpy())
    _, st = _compare.compare_step(w, ld, lt, roots, delta, g, check_verify=False)
    if test_id:
        record_parity(f"{test_id}[{delta}]", st)
    assert st["exact"] > 0 and st["near_tie"] + st["stop_near_tie"] <= 0.05 * (st["exact"] + 1)
    # and against the persistent build, bit for bit
    for f in FIELDS:
        a, b = getattr(want, f).cpu().numpy(), getattr(tree, f).cpu().numpy()
        assert np.array_equal(a, b, equal_nan=True), f
    return layers


@pytest.mark.parametrize("name,V,H", [("c1", 20000, 512), ("c2", 20000, 512), ("c4", 8200, 256), ("c3", 40008, 128), ("c5", 40008, 64)])
@pytest.mark.parametrize("delta", [NEG_INF, 0.2])
def test_reduced_tables(request, name, V, H, delta):
    _run(synth.WORKLOADS[name], delta, H=H, V=V, test_id=request.node.nodeid)


@pytest.mark.parametrize("n,k,D,B,V", [(1, 4, 5, 3, 512), (6, 1, 6, 3, 512), (5, 8, 3, 4, 8), (7, 3, 4, 2, 12), (10, 10, 6, 5, 104),
                                       (65, 4, 9, 2, 1024),
                                       # node budgets beyond 256: the larger layout of the layer team's scratch
                                       (300, 8, 6, 2, 2048), (1024, 32, 5, 1, 4096)])
def test_edge_sizes(request, n, k, D, B, V):
    w = synth.Workload("edge", B, V, n, k, D, 3.0, 1.1, 0.3, H=64, seed=n * 1000 + k)
    for delta in (NEG_INF, 0.1):
        _run(w, delta, test_id=request.node.nodeid)


def test_full_size_c4(request):
    assert _run(synth.WORKLOADS["c4"], NEG_INF, test_id=request.node.nodeid) == 10
