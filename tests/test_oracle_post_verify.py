"""Pins of the oracle's post-verification bookkeeping (dense mask, cache keep list)."""
import json
import os

import numpy as np

import oracle
from paper_2406_17276_b200 import synth

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_example_eq2_eq3.json")))


def test_hand_example():
    g = GOLD["n4"]; pv = GOLD["post_verify_n4"]
    dense = oracle.dense_mask_of(g["parent"], 4, 4)
    assert dense.tolist() == pv["dense_mask"]
    for case, want in zip(GOLD["verify_n4"], pv["kv"]):
        gather, kept = oracle.kv_keep_of(case["accept_nodes"] + [-1] * (3 - len(case["accept_nodes"])), case["accept_len"], 3)
        assert kept == want["kept"] and gather[:kept].tolist() == want["gather"] and (gather[kept:] == -1).all()


def _trees():
    w = synth.Workload("pv", 6, 512, 24, 5, 7, 3.0, 1.1, 0.3, H=64, seed=3)
    ld, lt = synth.make_tables(w)
    roots = synth.root_tokens(w.batch, w.V, 9)
    return w, oracle.table_step(ld, lt, roots, w.n, w.k, w.max_depth, 0.05)


def test_dense_mask_is_the_reachability_closure():
    """Independent definition: (I + adjacency)^n over booleans, plus the root column."""
    w, r = _trees()
    for b in range(w.batch):
        ns, n = int(r.n_sel[b]), w.n
        dense = oracle.dense_mask_of(r.parent[b], ns, n)
        adj = np.eye(n + 1, dtype=bool)
        for i in range(ns):
            adj[i + 1, r.parent[b, i] + 1 if r.parent[b, i] >= 0 else 0] = True      # node -> its parent (or the root)
        reach = adj.copy()
        for _ in range(n):
            reach = reach | ((reach.astype(np.int32) @ adj.astype(np.int32)) > 0)
        assert np.array_equal(dense.astype(bool), reach)
        # packed order puts ancestors first: lower triangular; a kept node sees itself, the root and depth-1 ancestors
        assert np.array_equal(np.tril(dense), dense)
        assert np.array_equal(dense[1:ns + 1].sum(1), r.depth[b, :ns] + 1)
        assert np.array_equal(dense[ns + 1:], np.eye(n + 1, dtype=np.uint8)[ns + 1:])


def test_dense_mask_agrees_with_the_bitmask():
    w, r = _trees()
    for b in range(w.batch):
        dense = oracle.dense_mask_of(r.parent[b], int(r.n_sel[b]), w.n)
        for i in range(int(r.n_sel[b])):
            bits = [(int(r.mask[b, i, j // 64]) >> (j % 64)) & 1 for j in range(w.n)]
            assert dense[i + 1, 1:].tolist() == bits


def test_kept_entries_follow_the_accepted_path():
    w, r = _trees()
    for b in range(w.batch):
        A = int(r.accept_len[b])
        gather, kept = oracle.kv_keep_of(r.accept_nodes[b], A, w.max_depth)
        assert kept == A and gather[0] == 0 and (gather[A:] == -1).all()
        for j in range(1, A):
            node = gather[j] - 1
            assert r.token[b, node] == r.accept_tokens[b, j - 1]                   # the kept node carries the accepted token
            assert r.parent[b, node] == gather[j - 1] - 1                           # and hangs under the previous kept position
        assert np.all(np.diff(gather[:A]) > 0)
