"""-m gpu: opt_tree_verify_static, the verification entry point for callers that cannot allocate.

Some users of this library may not call cudaMalloc at all once they are running (an engine whose memory
pool owns the device, a latency-critical loop that cannot afford an allocation's device-wide
synchronisation), so they cannot create a context.  The entry point keeps its scratch in an array inside
the library image instead.  Here it is driven through the C ABI with buffers that exist before the first
call, twice in a row on different inputs (the second call meets the first call's leftovers in the shared
array), and must reproduce opt_tree_verify exactly: every output is an integer.  The file sorts last so
that a run stopping at the first failure has already been through every other test.
"""
import math

import numpy as np
import pytest
import torch

from paper_2406_17276_b200 import binding, synth
from tests._gpu import dev_table

pytestmark = pytest.mark.gpu


def test_static_verify_matches_context_verify_on_two_calls_in_a_row():
    w = synth.Workload("noalloc", 6, 8200, 24, 6, 8, 3.0, 1.1, 0.3, H=128, seed=11)
    ld, lt = synth.make_tables(w)
    d_ld, d_lt = dev_table(ld), dev_table(lt)
    ot = binding.OptTree(w.V, w.H, w.n, w.k, w.max_depth, w.batch)
    cfg = binding.Config(w.V, w.H, w.n, w.k, w.max_depth, w.batch)
    i32 = dict(dtype=torch.int32, device="cuda")
    mine = (torch.empty(w.batch, **i32), torch.empty((w.batch, w.max_depth + 1), **i32),
            torch.empty((w.batch, w.max_depth), **i32), torch.empty(w.batch, **i32))
    status = torch.full((1,), 77, **i32)
    for call, seed in enumerate((3, 4)):
        roots = torch.from_numpy(synth.root_tokens(w.batch, w.V, seed)).cuda()
        tree = ot.build(d_ld, roots, -math.inf)
        ref = ot.verify(tree, d_lt, roots)
        for t in mine:
            t.fill_(-7)
        binding.verify_static(cfg, tree, d_lt, roots, mine, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert ot.device_status() == 0
        for name, a, b in zip(("accept_len", "accept_tokens", "accept_nodes", "next_root"), mine, ref):
            assert torch.equal(a, b), f"call {call}: {name} differs"
        assert int(mine[0].min()) >= 1


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
