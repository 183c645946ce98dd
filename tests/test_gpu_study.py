"""-m gpu: the acceptance-length study (adaptive tree against fixed trees on the same roots) reports what an
independent evaluation on the host finds: the oracle for the adaptive tree, NumPy definitions for the
sequence draft and the complete binary / 4-ary trees."""
import math

import numpy as np
import pytest

import oracle
from paper_2406_17276_b200 import study, synth
from tests import _defs

pytestmark = pytest.mark.gpu


def _fixed_tree_stats(ld, lt, root, b, n):
    """E(A) (sum of path values) and acceptance length of the complete b-ary tree cut off at n nodes."""
    depth, total = 0, 0
    while total < n:
        depth += 1
        total += b ** depth
    nodes = _defs.full_tree(ld, root, b, depth)[:n]        # breadth first: level by level, parents in order, siblings by rank
    paths = {nd[0] for nd in nodes}
    chain = _defs.target_chain(lt, root, depth + 1)
    hits = 0
    while hits < depth and tuple(chain[:hits + 1]) in paths:
        hits += 1
    return sum(nd[1] for nd in nodes), hits + 1


def test_study_agrees_with_host_side_definitions():
    steps = 4
    res, first = study.run("c1", steps, keep_first=steps)
    w, n = first["w"], first["n"]
    ld, lt = first["tables"]
    for s in range(steps):
        roots = first["roots"][s]
        o = oracle.table_step(ld, lt, roots, n, w.k, w.max_depth, -math.inf)
        for b in range(w.batch):
            if o.min_gap[b] >= 1e-6:
                assert first["A_shapes"]["opt_tree"][s, b] == o.accept_len[b]
                assert first["E_shapes"]["opt_tree"][s, b] == pytest.approx(o.expected_len[b], rel=1e-5)
            for shape, br in (("binary", 2), ("4-ary", 4), ("sequence", 1)):
                e, a = _fixed_tree_stats(ld, lt, int(roots[b]), br, n)
                assert first["A_shapes"][shape][s, b] == a, (shape, s, b)
                assert first["E_shapes"][shape][s, b] == pytest.approx(e, rel=1e-5), (shape, s, b)
        deep = oracle.table_step(ld, lt, roots, n, w.k, min(n, 500), 0.0)      # depth limited by n alone, threshold 0
        for b in range(w.batch):
            if deep.min_gap[b] >= 1e-6 and deep.stop_margin[b] >= 1e-5:
                assert first["A_shapes"]["opt_tree_depth_n"][s, b] == deep.accept_len[b]
                assert first["E_shapes"]["opt_tree_depth_n"][s, b] == pytest.approx(deep.expected_len[b], rel=1e-5)
    sh = res["shapes"]
    assert sh["opt_tree"]["mean_expected_length_plus_1"] >= sh["binary"]["mean_expected_length_plus_1"] - 1e-9
    assert sh["opt_tree"]["mean_expected_length_plus_1"] >= sh["4-ary"]["mean_expected_length_plus_1"] - 1e-9
    # (the sequence draft may go deeper than the workload's depth limit; against the tree limited by n alone the bound holds)
    assert sh["opt_tree_depth_n"]["mean_expected_length_plus_1"] >= sh["sequence"]["mean_expected_length_plus_1"] - 1e-6
    h = np.array(res["hist_rows_rounded_EA_plus_1_cols_A"])
    assert h.sum() == steps * w.batch
