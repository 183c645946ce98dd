"""No GPU: the benchmark's host-side arithmetic (row counts behind the algorithmic bytes, the classification of
the checked step against the oracle, the recorded-traffic lookup)."""
import math
import types

import numpy as np

import bench
from paper_2406_17276_b200 import synth


def test_logical_rows_is_the_root_row_the_first_layer_and_full_layers():
    w = synth.WORKLOADS["c4"]                       # n = 64, k = 10, depth 10
    assert bench.logical_rows(w, [10]) == 1 + 10 + 8 * 64 == 523
    assert bench.logical_rows(w, [1]) == 1 and bench.logical_rows(w, [2]) == 11 and bench.logical_rows(w, [3]) == 75
    assert bench.logical_rows(w, [10] * 32) == 32 * 523
    c1 = synth.WORKLOADS["c1"]                      # n = k = 10: the first layer is as wide as the others
    assert bench.logical_rows(c1, [6]) == 1 + 10 + 4 * 10


def _fake(B, n, D):
    g = dict(token=np.zeros((B, n), np.int32), parent=np.full((B, n), -1, np.int32), depth=np.ones((B, n), np.int32),
             n_sel=np.full(B, n, np.int32), depth_reached=np.full(B, D, np.int32), mask=np.zeros((B, n, 1), np.uint64),
             position_ids=np.ones((B, n), np.int32), accept_len=np.ones(B, np.int32), accept_tokens=np.zeros((B, D + 1), np.int32),
             accept_nodes=np.full((B, D), -1, np.int32), next_root=np.zeros(B, np.int32),
             phat=np.full((B, n), 0.5), expected_len=np.full(B, 0.5 * n))
    o = types.SimpleNamespace(**{k: v.copy() for k, v in g.items()}, min_gap=np.full(B, 0.3))
    return g, o


def test_parity_counts_sorts_sequences_into_exact_near_tie_and_mismatch():
    g, o = _fake(4, 3, 2)
    o.token[1, 0] = 7; o.min_gap[1] = 1e-9          # differs at a near tie: exempt, counted
    o.token[2, 0] = 7                                # differs with a wide gap: a mismatch
    g["phat"][3, 1] *= 1.0 + 5e-5                    # integers agree, a path value is off by more than 1e-5
    r = bench.parity_counts(g, o)
    assert (r["exact"], r["near_tie"], r["mismatch"], r["sequences"]) == (2, 1, 2, 4)
    assert r["max_phat_rel"] > 1e-5
    g2, o2 = _fake(3, 2, 2)
    r2 = bench.parity_counts(g2, o2)
    assert (r2["exact"], r2["near_tie"], r2["mismatch"]) == (3, 0, 0) and r2["max_phat_rel"] == 0.0


def test_recorded_traffic_is_dropped_when_sources_or_threshold_differ(monkeypatch):
    key = ("c4", 4096)
    assert key in bench.NCU_TRAFFIC
    monkeypatch.setitem(bench.NCU_TRAFFIC, key, {"bytes": 1.0, "csrc_sha256": bench._csrc_digest()})
    assert bench._ncu_traffic("c4", 4096, -math.inf) == 1.0
    assert bench._ncu_traffic("c4", 4096, 0.2) is None               # counters were taken with the threshold off
    assert bench._ncu_traffic("c4", 12345, -math.inf) is None
    monkeypatch.setitem(bench.NCU_TRAFFIC, key, {"bytes": 1.0, "csrc_sha256": "0" * 64})
    assert bench._ncu_traffic("c4", 4096, -math.inf) is None         # the kernels changed since
