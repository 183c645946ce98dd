"""-m gpu: every kind of bounded device-side wait gives up with a timeout status instead of hanging.

opt_tree_selftest_waits enters each wait on something nobody completes (a fresh shared-memory barrier,
words that stay zero, a row source that never has a row) with a limit of microseconds; the kernel must
end and every wait must have recorded OPT_TREE_ERR_TIMEOUT in its own status word.  The context stays
usable afterwards.
"""
import math

import numpy as np
import pytest
import torch

from paper_2406_17276_b200 import binding, synth
from tests._gpu import dev_table

pytestmark = pytest.mark.gpu


def test_every_bounded_wait_runs_out_and_reports_a_timeout():
    w = synth.Workload("waits", 2, 512, 8, 4, 4, 3.0, 1.1, 0.3, H=16, seed=2)
    ld, _ = synth.make_tables(w)
    ot = binding.OptTree(w.V, w.H, w.n, w.k, w.max_depth, w.batch)
    res = ot.selftest_waits()
    torch.cuda.synchronize()
    assert res.cpu().tolist() == [binding.ERR_TIMEOUT] * 5
    assert ot.device_status() == 0                                   # the context's own word is untouched
    # the context still builds trees
    tree = ot.build(dev_table(ld), torch.from_numpy(synth.root_tokens(2, w.V, 1)).cuda(), -math.inf)
    torch.cuda.synchronize()
    assert ot.device_status() == 0 and int(tree.n_sel.min()) == w.n
