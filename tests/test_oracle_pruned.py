"""The pruned draft (only layer nodes still among the n largest are expanded) gives the same tree.

Theorem 1 (a node's path value is below its parent's) is the reason; these tests check the claim
on the oracle itself, over random tables, thresholds and shapes, before any GPU code relies on it.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2406_17276_b200 import synth

FIELDS = ("token", "parent", "depth", "phat", "n_sel", "depth_reached", "expected_len", "esub_trace")


@pytest.mark.parametrize("n,k,D,V,sigma", [(10, 10, 6, 512, 3.0), (24, 5, 8, 512, 1.0), (64, 10, 10, 2048, 3.0), (7, 3, 5, 64, 0.5),
                                           (16, 16, 12, 256, 4.0), (1, 4, 5, 128, 3.0), (6, 1, 6, 128, 3.0), (40, 8, 3, 512, 2.0)])
@pytest.mark.parametrize("delta", [-math.inf, 0.0, 0.05, 0.3])
def test_pruned_equals_full(n, k, D, V, sigma, delta):
    w = synth.Workload("pr", 6, V, n, k, D, sigma, 1.1, 0.0, H=64, seed=n * 100 + k)
    ld, _ = synth.make_tables(w)
    roots = synth.root_tokens(w.batch, V, 17)
    full, rows_full = oracle.table_build_rows(ld, roots, n, k, D, delta, prune=False)
    pruned, rows_pruned = oracle.table_build_rows(ld, roots, n, k, D, delta, prune=True)
    for f in FIELDS:
        assert np.array_equal(full[f], pruned[f]), f
    assert np.all(rows_pruned <= rows_full)


def test_full_variant_is_the_ordinary_build():
    w = synth.Workload("pr", 4, 512, 24, 5, 8, 3.0, 1.1, 0.0, H=64, seed=5)
    ld, lt = synth.make_tables(w)
    roots = synth.root_tokens(w.batch, w.V, 3)
    full, rows = oracle.table_build_rows(ld, roots, w.n, w.k, w.max_depth, 0.05, prune=False)
    r = oracle.table_step(ld, lt, roots, w.n, w.k, w.max_depth, 0.05)
    for f in FIELDS:
        assert np.array_equal(full[f], getattr(r, f)), f
    # rows of the full build: the root, then every node of every drafted layer but the last
    for b in range(w.batch):
        d = int(r.depth_reached[b])
        assert rows[b] == 1 + (min(w.n, w.k) if d >= 2 else 0) + max(0, d - 2) * w.n


def test_pruning_saves_rows_on_the_benchmark_shape():
    w = synth.WORKLOADS["c4"]
    ld, _ = synth.make_tables(w, H=256, V=4096)
    roots = synth.root_tokens(4, 4096, 3)
    _, rows_full = oracle.table_build_rows(ld, roots, w.n, w.k, w.max_depth, -math.inf, prune=False)
    _, rows_pruned = oracle.table_build_rows(ld, roots, w.n, w.k, w.max_depth, -math.inf, prune=True)
    assert rows_pruned.sum() < 0.6 * rows_full.sum()
