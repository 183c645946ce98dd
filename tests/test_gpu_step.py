"""-m gpu: whole decoding steps (build, mask, verify) through the C ABI against the oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2406_17276_b200 import binding, synth
from tests import _compare
from tests._gpu import add_stats, dev_table, gpu_step, new_totals, record_parity

pytestmark = pytest.mark.gpu
NEG_INF = -math.inf


def _run(w, deltas, steps=1, H=None, V=None, chain=False):
    ld, lt = synth.make_tables(w, H=H, V=V)
    Hh, Vv = ld.shape
    ot = binding.OptTree(Vv, Hh, w.n, w.k, w.max_depth, w.batch)
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    memo = oracle.Memo(w.k, cap=4 * Hh)
    total = new_totals()
    for delta in deltas:
        roots = synth.root_tokens(w.batch, Vv, w.seed + 1)
        base = np.arange(w.batch, dtype=np.int32) * 7 + 3
        for _ in range(steps):
            g = gpu_step(ot, d_ld, d_lt, roots, delta, base)
            o, st = _compare.compare_step(w, ld, lt, roots, delta, g, base_pos=base, memo=memo)
            add_stats(total, st)
            roots = o.next_root.copy()           # the oracle's token feeds the next step (Algorithm 2, Concat)
            base = base + o.accept_len
    return total


@pytest.mark.parametrize("name,V,H", [("c1", 20000, 512), ("c2", 20000, 512), ("c4", 20000, 512), ("c4", 8200, 256),
                                      ("c3", 40008, 128), ("c5", 40008, 128)])
def test_reduced_tables_all_thresholds(request, name, V, H):
    w = synth.WORKLOADS[name]
    t = _run(w, [NEG_INF, 0.0, 0.2, 0.7], steps=3, H=H, V=V)
    record_parity(request.node.nodeid, t)
    assert t["exact"] > 0 and t["near_tie"] + t["stop_near_tie"] <= 0.05 * (t["exact"] + 1)


@pytest.mark.parametrize("name,steps", [("c1", 20), ("c2", 10), ("c3", 3), ("c4", 3), ("c5", 1)])
def test_full_size_configurations(request, name, steps):
    w = synth.WORKLOADS[name]
    t = _run(w, [NEG_INF] if name == "c5" else [NEG_INF, 0.2], steps=steps)
    record_parity(request.node.nodeid, t)
    assert t["exact"] > 0 and t["near_tie"] + t["stop_near_tie"] <= 0.05 * (t["exact"] + 1)


@pytest.mark.parametrize("n,k,D,B,V", [(1, 4, 5, 3, 512), (6, 1, 6, 3, 512), (256, 32, 20, 2, 4096), (5, 8, 3, 4, 8),
                                       (7, 3, 4, 2, 12), (64, 10, 10, 1, 32000), (10, 10, 6, 5, 100),
                                       # more sequences than CTAs (a layer warp follows several), and more than
                                       # four per CTA (they are then followed in waves)
                                       (8, 4, 4, 300, 512), (6, 3, 3, 700, 256)])
def test_degenerate_and_maximum_sizes(request, n, k, D, B, V):
    w = synth.Workload("edge", B, V, n, k, D, 3.0, 1.1, 0.3, H=64, seed=n * 1000 + k)
    t = _run(w, [NEG_INF, 0.1], steps=2)
    record_parity(request.node.nodeid, t)
    assert t["exact"] > 0 and t["near_tie"] + t["stop_near_tie"] <= 0.05 * (t["exact"] + 1)


@pytest.mark.parametrize("n,k,D,B", [(512, 16, 10, 4), (512, 32, 8, 3), (1000, 16, 8, 3), (1000, 32, 6, 2), (1024, 32, 12, 2), (300, 4, 24, 1)])
def test_node_budgets_beyond_256(request, n, k, D, B):
    """Trees of several hundred to a thousand nodes (the paper's Section 4.3 grows its trees past 500 nodes):
    V = 32000, a table of 512 rows so that the oracle's row memo keeps the comparison short."""
    w = synth.Workload("large_n", B, 32000, n, k, D, 3.0, 1.1, 0.2, H=512, seed=n + k)
    t = _run(w, [NEG_INF, 0.05], steps=2)
    record_parity(request.node.nodeid, t)
    assert t["exact"] > 0 and t["near_tie"] + t["stop_near_tie"] <= 0.05 * (t["exact"] + 1)


@pytest.mark.parametrize("name,V,H,steps,delta", [("c4", 20000, 512, 25, NEG_INF), ("c2", 20000, 512, 60, 0.2), ("c1", 32000, 4096, 100, NEG_INF)])
def test_free_running_chain_leaves_the_oracle_only_at_a_near_tie(request, name, V, H, steps, delta):
    """The library decodes on its own: every step starts from the token its own verification accepted last
    (Algorithm 2's Concat).  The oracle runs its own chain from the same first roots.  As long as a sequence
    has agreed in every earlier step both sides see the same root; the first step whose integer outputs differ
    must be one where the oracle reports a selection boundary closer than 1e-6 (or a loop test within
    tolerance), and such sequences are counted."""
    w = synth.WORKLOADS[name]
    ld, lt = synth.make_tables(w, H=H, V=V)
    ot = binding.OptTree(V, H, w.n, w.k, w.max_depth, w.batch)
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    memo = oracle.Memo(w.k, cap=4 * H)
    g_roots = synth.root_tokens(w.batch, V, w.seed + 3)
    o_roots = g_roots.copy()
    in_sync = np.ones(w.batch, bool)
    st = new_totals()
    for _ in range(steps):
        g = gpu_step(ot, d_ld, d_lt, g_roots, delta)
        o = oracle.table_step(ld, lt, o_roots, w.n, w.k, w.max_depth, float(np.float32(delta)), memo=memo)
        for b in np.nonzero(in_sync)[0]:
            assert g_roots[b] == o_roots[b]
            ob = _compare._slice(o, b)
            if _compare._ints_equal(g, ob, b, True):
                st["exact"] += 1
                _compare._check_floats(g, ob, b, st)
            else:
                near = o.min_gap[b] < _compare.GAP_EXEMPT or o.stop_margin[b] < _compare.FLOAT_RTOL * max(1.0, o.expected_len[b])
                assert near, f"sequence {b} left the oracle's chain at a step whose smallest gap is {o.min_gap[b]:.3e}"
                st["near_tie"] += 1
                in_sync[b] = False
        g_roots, o_roots = g["next_root"].copy(), o.next_root.copy()
    record_parity(request.node.nodeid, st)
    assert in_sync.sum() >= 0.9 * w.batch


def test_two_runs_are_bit_identical():
    w = synth.WORKLOADS["c4"]
    ld, lt = synth.make_tables(w, H=256, V=20000)
    ot = binding.OptTree(20000, 256, w.n, w.k, w.max_depth, w.batch)
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    roots = synth.root_tokens(w.batch, 20000, 9)
    a = gpu_step(ot, d_ld, d_lt, roots, 0.2)
    b = gpu_step(ot, d_ld, d_lt, roots, 0.2)
    for f in a:
        assert np.array_equal(a[f], b[f], equal_nan=True), f


def test_identical_tables_accept_at_least_two_tokens():
    w = synth.Workload("same", 8, 8200, 24, 6, 8, 3.0, 1.1, 0.0, H=128, seed=77)
    ld, _ = synth.make_tables(w)
    ot = binding.OptTree(w.V, w.H, w.n, w.k, w.max_depth, w.batch)
    d = dev_table(ld)
    g = gpu_step(ot, d, d, synth.root_tokens(8, w.V, 1), NEG_INF)
    assert np.all(g["accept_len"] >= 2)


def test_host_buffer_step_matches_device_path():
    w = synth.WORKLOADS["c4"]
    ld, lt = synth.make_tables(w, H=256, V=20000)
    ot = binding.OptTree(20000, 256, w.n, w.k, w.max_depth, w.batch)
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    roots = synth.root_tokens(w.batch, 20000, 4)
    base = np.arange(w.batch, dtype=np.int32)
    g = gpu_step(ot, d_ld, d_lt, roots, 0.2, base)
    ho = ot.alloc_host_out(w.batch)
    ot.step_host(d_ld, d_lt, torch.from_numpy(roots).pin_memory(), torch.from_numpy(base).pin_memory(), 0.2, ho)
    for f, t in ho.items():
        assert np.array_equal(t.numpy(), g[f]), f


def test_argument_checks_return_status_codes():
    with pytest.raises(binding.OptTreeError) as e:
        binding.OptTree(32000, 64, 1025, 10, 10, 1)
    assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.OptTreeError) as e:
        binding.OptTree(32000, 64, 64, 33, 10, 1)
    assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.OptTreeError) as e:
        binding.OptTree(8, 64, 4, 9, 3, 1)                   # k > V
    assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.OptTreeError) as e:
        binding.OptTree(0, 64, 4, 2, 3, 1)
    assert e.value.code == binding.ERR_INVALID_ARG
    ot = binding.OptTree(512, 64, 8, 4, 4, 2)
    tab = torch.zeros((64, 512), dtype=torch.int16, device="cuda")
    with pytest.raises(binding.OptTreeError) as e:
        ot.build(tab, torch.zeros(3, dtype=torch.int32, device="cuda"), 0.0)     # B > max_batch
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.OptTreeError) as e:
        ot.build(tab, torch.zeros(2, dtype=torch.int32, device="cuda"), float("nan"))
    assert e.value.code == binding.ERR_INVALID_ARG


def test_exact_ties_are_broken_by_index(request):
    """Every row gives k tokens the same logit and masks the rest, so every child has probability
    exactly 1/k, all candidates of a layer have the same path value, and the selection is decided by
    the tie rules alone (depth, then candidate index)."""
    B, V, H, n, k, D = 4, 2048, 64, 64, 10, 6
    w = synth.Workload("ties", B, V, n, k, D, 3.0, 1.1, 0.0, H=H, seed=5)
    rng = np.random.default_rng(11)
    ld = np.full((H, V), 0xFF80, np.uint16)                       # -inf
    for h in range(H):
        ld[h, rng.choice(V, k, replace=False)] = 0x3F80           # 1.0 in bf16
    ot = binding.OptTree(V, H, n, k, D, B)
    d = dev_table(ld)
    roots = synth.root_tokens(B, V, 3)
    for delta in (NEG_INF, 0.05):
        g = gpu_step(ot, d, d, roots, delta)
        o, st = _compare.compare_step(w, ld, ld, roots, delta, g)
        record_parity(f"{request.node.nodeid}[{delta}]", st)
        assert st["exact"] == B and st["near_tie"] == 0, st
