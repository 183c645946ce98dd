"""-m gpu: opt_tree_verify_static, the verification entry point for callers that cannot allocate.

Some users of this library may not call cudaMalloc at all once they are running (an engine whose memory
pool owns the device, a latency-critical loop that cannot afford an allocation's device-wide
synchronisation), so they cannot create a context.  The entry point keeps its scratch in an array inside
the library image instead.  Here it is driven through the C ABI with buffers that exist before the first
call, twice in a row on different inputs (the second call meets the first call's leftovers in the shared
array), and must reproduce opt_tree_verify and the oracle's greedy walk exactly: every output is an
integer.  The file sorts last so that a run stopping at the first failure has already been through every
other test.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2406_17276_b200 import binding, synth
from tests._gpu import dev_table, poison

pytestmark = pytest.mark.gpu
NAMES = ("accept_len", "accept_tokens", "accept_nodes", "next_root")


def _two_calls(w, max_batch_field, H=None, V=None, unaligned=False):
    ld, lt = synth.make_tables(w, H=H, V=V)
    Hh, Vv = ld.shape
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    ot = binding.OptTree(Vv, Hh, w.n, w.k, w.max_depth, w.batch)
    cfg = binding.Config(Vv, Hh, w.n, w.k, w.max_depth, max_batch_field)
    i32 = dict(dtype=torch.int32, device="cuda")
    mine = (torch.empty(w.batch, **i32), torch.empty((w.batch, w.max_depth + 1), **i32),
            torch.empty((w.batch, w.max_depth), **i32), torch.empty(w.batch, **i32))
    status = torch.full((1,), 77, **i32)
    for call, seed in enumerate((3, 4)):
        roots_np = synth.root_tokens(w.batch, Vv, seed)
        roots = torch.from_numpy(roots_np).cuda()
        tree = ot.build(d_ld, roots, -math.inf)
        ref = ot.verify(tree, d_lt, roots)
        poison(*mine)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        reserved_before = torch.cuda.memory_reserved()
        binding.verify_static(cfg, tree, d_lt, roots, mine, status)
        torch.cuda.synchronize()
        # nothing was allocated through torch by either call, and the device's free memory is the same before
        # and after the second one (the first may make the driver load code it has not used yet)
        assert torch.cuda.memory_reserved() == reserved_before
        assert call == 0 or torch.cuda.mem_get_info()[0] == free_before
        assert int(status.item()) == 0
        assert ot.device_status() == 0
        for name, a, b in zip(NAMES, mine, ref):
            assert torch.equal(a, b), f"call {call}: {name} differs from opt_tree_verify"
        # and against the oracle's walk on the same trees (integers: exact)
        t = {f: getattr(tree, f).cpu().numpy() for f in ("token", "parent", "depth", "n_sel")}
        for b in range(w.batch):

            def target(root, path, _lt=lt, _H=Hh):
                tok, dep = (root, 0) if len(path) == 0 else (path[-1], len(path))
                return synth.bf16_bits_to_f32(_lt[(tok * 31 + dep) % _H]).astype(np.float64)
            o = oracle.verify_cb(target, int(roots_np[b]), Vv, int(t["n_sel"][b]), w.max_depth, t["token"][b], t["parent"][b], t["depth"][b])
            assert int(mine[0][b]) == o["accept_len"], f"call {call}, sequence {b}: accept_len differs from the oracle"
            assert np.array_equal(mine[1][b].cpu().numpy(), o["accept_tokens"])
            assert np.array_equal(mine[2][b].cpu().numpy(), o["accept_nodes"])
            assert int(mine[3][b]) == o["next_root"]
        assert int(mine[0].min()) >= 1


def test_static_verify_matches_context_verify_on_two_calls_in_a_row():
    _two_calls(synth.Workload("noalloc", 6, 8200, 24, 6, 8, 3.0, 1.1, 0.3, H=128, seed=11), max_batch_field=6)


def test_static_verify_ignores_the_max_batch_field_and_takes_any_vocabulary_size():
    # max_batch left at zero; V not a multiple of 8, so rows are not 16-byte aligned (the scalar path)
    _two_calls(synth.Workload("noalloc", 3, 1001, 12, 4, 5, 3.0, 1.1, 0.3, H=32, seed=12), max_batch_field=0)


def test_static_verify_at_the_limits_of_its_array():
    _two_calls(synth.Workload("noalloc", 64, 2048, 256, 32, 6, 2.5, 1.05, 0.3, H=64, seed=13), max_batch_field=64)


def test_static_verify_rejects_sizes_beyond_its_array():
    w = synth.Workload("noalloc", 2, 512, 8, 4, 4, 3.0, 1.1, 0.3, H=16, seed=2)
    ld, lt = synth.make_tables(w)
    ot = binding.OptTree(w.V, w.H, w.n, w.k, w.max_depth, 128)
    i32 = dict(dtype=torch.int32, device="cuda")
    B = 65                                                    # one more than OPT_TREE_STATIC_MAX_BATCH
    roots = torch.zeros(B, **i32)
    tree = ot.build(dev_table(ld), roots, -math.inf)
    out = (torch.empty(B, **i32), torch.empty((B, w.max_depth + 1), **i32), torch.empty((B, w.max_depth), **i32),
           torch.empty(B, **i32))
    with pytest.raises(binding.OptTreeError) as e:
        binding.verify_static(binding.Config(w.V, w.H, w.n, w.k, w.max_depth, 128), tree, dev_table(lt), roots, out)
    assert e.value.code == binding.ERR_UNSUPPORTED
    torch.cuda.synchronize()
