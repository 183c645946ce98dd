"""-m gpu: the bookkeeping after verification (dense mask, cache keep list) against the oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2406_17276_b200 import binding, synth
from tests._gpu import dev_table

pytestmark = pytest.mark.gpu


def _check(w, delta, H=None, V=None):
    ld, lt = synth.make_tables(w, H=H, V=V)
    Hh, Vv = ld.shape
    ot = binding.OptTree(Vv, Hh, w.n, w.k, w.max_depth, w.batch)
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    roots = synth.root_tokens(w.batch, Vv, w.seed + 2)
    r = torch.from_numpy(roots).cuda()
    tree = ot.build(d_ld, r, delta)
    mask, _ = ot.mask(tree, None)
    al, at, an, nr = ot.verify(tree, d_lt, r)
    dense, gather, keep = ot.post_verify(tree, mask, al, an)
    torch.cuda.synchronize()
    assert ot.device_status() == 0
    parent = tree.parent.cpu().numpy(); n_sel = tree.n_sel.cpu().numpy()
    al_h, an_h = al.cpu().numpy(), an.cpu().numpy()
    dense, gather, keep = dense.cpu().numpy(), gather.cpu().numpy(), keep.cpu().numpy()
    for b in range(w.batch):
        # the oracle works on the tree and the acceptance the device produced (those have their own parity tests)
        want = oracle.dense_mask_of(parent[b], int(n_sel[b]), w.n)
        assert np.array_equal(dense[b], want), b
        g, kept = oracle.kv_keep_of(an_h[b], int(al_h[b]), w.max_depth)
        assert keep[b] == kept and np.array_equal(gather[b], g), b


@pytest.mark.parametrize("name,V,H,delta", [("c4", 20000, 256, -math.inf), ("c4", 8200, 128, 0.3), ("c2", 20000, 256, 0.7),
                                           ("c5", 40008, 64, -math.inf)])
def test_reduced_tables(name, V, H, delta):
    _check(synth.WORKLOADS[name], delta, H=H, V=V)


@pytest.mark.parametrize("n,k,D,B,V", [(1, 4, 5, 3, 512), (6, 1, 6, 3, 512), (256, 32, 20, 2, 4096), (5, 8, 3, 4, 8),
                                       (65, 4, 9, 2, 1024), (128, 6, 7, 2, 2048)])
def test_edge_sizes(n, k, D, B, V):
    _check(synth.Workload("edge", B, V, n, k, D, 3.0, 1.1, 0.3, H=64, seed=n * 31 + k), 0.05)


def test_full_size_c4():
    _check(synth.WORKLOADS["c4"], -math.inf)


def test_argument_checks():
    w = synth.WORKLOADS["c1"]
    ot = binding.OptTree(512, 64, w.n, w.k, w.max_depth, 1)
    tree = ot.alloc_tree(1, trace=False)
    with pytest.raises(Exception):
        ot.post_verify(tree, None, torch.zeros(1, dtype=torch.int32, device="cuda"), torch.zeros((1, w.max_depth), dtype=torch.int32, device="cuda"))
