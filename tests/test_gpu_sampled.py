"""-m gpu: verification with sampling against the oracle's same rule and the same uniforms."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2406_17276_b200 import binding, synth
from tests._gpu import dev_table, poisoned_verify_out, record_parity

pytestmark = pytest.mark.gpu
MARGIN = 2e-6         # a draw may fall the other way only where u*S sits this close (relative to S) to a running sum:
                      # the library adds up each 512-logit segment in single precision (a few 1e-7 of S at worst)


def _run(w, taus, H=None, V=None, steps=2, test_id=None):
    ld, lt = synth.make_tables(w, H=H, V=V)
    Hh, Vv = ld.shape
    ot = binding.OptTree(Vv, Hh, w.n, w.k, w.max_depth, w.batch)
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    roots = synth.root_tokens(w.batch, Vv, w.seed + 8)
    exact = near = 0
    for tau in taus:
        r = torch.from_numpy(roots).cuda()
        tree = ot.build(d_ld, r, -math.inf)
        for step in range(steps):
            al, at, an, nr = ot.verify_sampled(tree, d_lt, r, tau, 1234, step, poisoned_verify_out(ot, w.batch))
            torch.cuda.synchronize()
            assert ot.device_status() == 0
            o = oracle.table_verify_sampled(lt, roots, tree.token.cpu().numpy(), tree.parent.cpu().numpy(), tree.depth.cpu().numpy(),
                                            tree.n_sel.cpu().numpy(), w.max_depth, tau, 1234, step)
            g = dict(accept_len=al.cpu().numpy(), accept_tokens=at.cpu().numpy(), accept_nodes=an.cpu().numpy(), next_root=nr.cpu().numpy())
            for b in range(w.batch):
                same = all(np.array_equal(g[f][b], o[f][b]) for f in g)
                if same:
                    exact += 1
                else:
                    assert o["min_margin"][b] < MARGIN, (b, tau, step, o["min_margin"][b], g["accept_tokens"][b], o["accept_tokens"][b])
                    near += 1
    if test_id:
        record_parity(test_id, dict(exact=exact, near_tie=near, stop_near_tie=0, max_phat_rel=0.0, max_elen_rel=0.0))
    assert exact > 0 and near <= 0.02 * (exact + 1)
    return exact, near


@pytest.mark.parametrize("name,V,H", [("c1", 20000, 256), ("c4", 8200, 128), ("c2", 20000, 256), ("c3", 40008, 64)])
def test_reduced_tables(request, name, V, H):
    _run(synth.WORKLOADS[name], [1.0, 0.5, 2.0], H=H, V=V, test_id=request.node.nodeid)


@pytest.mark.parametrize("n,k,D,B,V", [(1, 4, 5, 3, 512), (6, 1, 6, 3, 512), (5, 8, 3, 4, 8), (7, 3, 4, 2, 12), (64, 10, 10, 2, 4099)])
def test_edge_sizes(request, n, k, D, B, V):
    _run(synth.Workload("edge", B, V, n, k, D, 3.0, 1.1, 0.3, H=64, seed=n * 1000 + k), [1.0, 0.3], test_id=request.node.nodeid)


def test_full_size_c4(request):
    _run(synth.WORKLOADS["c4"], [1.0], steps=1, test_id=request.node.nodeid)


def test_low_temperature_is_the_greedy_walk():
    w = synth.Workload("lt", 8, 8200, 24, 6, 8, 3.0, 1.1, 0.3, H=128, seed=21)
    ld, lt = synth.make_tables(w)
    ot = binding.OptTree(w.V, w.H, w.n, w.k, w.max_depth, w.batch)
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    r = torch.from_numpy(synth.root_tokens(w.batch, w.V, 3)).cuda()
    tree = ot.build(d_ld, r, -math.inf)
    greedy = ot.verify(tree, d_lt, r)
    sampled = ot.verify_sampled(tree, d_lt, r, 1e-4, 5, 0)
    torch.cuda.synchronize()
    for a, b in zip(greedy, sampled):
        assert torch.equal(a, b)


def test_rejects_bad_temperature():
    w = synth.WORKLOADS["c1"]
    ot = binding.OptTree(512, 64, w.n, w.k, w.max_depth, 1)
    tree = ot.alloc_tree(1, trace=False)
    t = torch.zeros((64, 512), dtype=torch.int16, device="cuda")
    r = torch.zeros(1, dtype=torch.int32, device="cuda")
    for tau in (0.0, -1.0, float("nan")):
        with pytest.raises(Exception):
            ot.verify_sampled(tree, t, r, tau, 1, 0)
