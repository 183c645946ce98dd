"""Pins: theorems and special cases the paper fixes (no GPU)."""
import math

import numpy as np
import pytest

import oracle
from tests import _defs

NEG_INF = float("-inf")


def _build(tab, roots, n, k, D, delta=NEG_INF):
    return oracle.table_step(tab, None, np.asarray(roots, np.int32), n, k, D, delta)


@pytest.fixture(scope="module")
def tab():
    return _defs.small_table(256, 512, 7)


def test_theorem1_descendants_never_exceed_ancestors(tab):
    r = _build(tab, range(16), 24, 6, 8)
    for b in range(16):
        for i in range(r.n_sel[b]):
            p = r.parent[b, i]
            if p >= 0:
                assert r.phat[b, i] <= r.phat[b, p]
                assert r.phat[b, i] > 0.0


def test_closure_selected_nodes_form_a_rooted_subtree(tab):
    r = _build(tab, range(16), 24, 6, 8)
    for b in range(16):
        ns = r.n_sel[b]
        for i in range(ns):
            p = r.parent[b, i]
            assert -1 <= p < i                           # parent kept and packed earlier
            assert r.depth[b, i] == (1 if p < 0 else r.depth[b, p] + 1)
        assert np.all(r.token[b, ns:] == -1) and np.all(r.phat[b, ns:] == 0.0)


def test_theorem2_esub_non_decreasing_in_drafting_steps(tab):
    r = _build(tab, range(16), 24, 6, 8)
    for b in range(16):
        tr = r.esub_trace[b, :r.depth_reached[b]]
        assert np.all(np.diff(tr) >= 0.0)
        assert abs(tr[-1] - r.expected_len[b]) < 1e-12
        assert np.all(tr <= np.arange(1, len(tr) + 1) + 1e-12)   # each layer's path values sum to <= 1


def test_expected_len_non_decreasing_in_n(tab):
    prev = np.zeros(4)
    for n in range(1, 13):
        r = _build(tab, range(4), n, 12, 5)             # k >= n_max, threshold off, same depth
        assert np.all(r.expected_len >= prev - 1e-15)
        prev = r.expected_len.copy()


def test_expected_len_is_sum_of_path_values_eq3(tab):
    r = _build(tab, range(8), 20, 5, 6)
    for b in range(8):
        assert abs(r.phat[b, :r.n_sel[b]].sum() - r.expected_len[b]) < 1e-12


def test_path_values_are_products_of_numpy_probabilities_eq2(tab):
    r = _build(tab, [3, 99], 12, 4, 5)
    for b, root in enumerate([3, 99]):
        for i, path in enumerate(_defs.paths_of(r.token[b], r.parent[b], r.n_sel[b])):
            ph, tok, dep = 1.0, root, 0
            for t in path:
                _x, p = _defs.np_row_probs(tab, tok, dep)
                ph *= p[t]; tok, dep = t, dep + 1
            assert abs(ph - r.phat[b, i]) <= 1e-12 * ph


def test_k1_gives_the_greedy_chain(tab):
    D = 6
    r = _build(tab, [5], 6, 1, D)
    tok, dep, ph, want_tok, want_ph = 5, 0, 1.0, [], []
    for _ in range(D):
        x, p = _defs.np_row_probs(tab, tok, dep)
        j = int(_defs.np_topk(x, 1)[0])
        ph *= p[j]; tok, dep = j, dep + 1
        want_tok.append(j); want_ph.append(ph)
    assert r.token[0].tolist() == want_tok
    assert r.parent[0].tolist() == [-1, 0, 1, 2, 3, 4]
    np.testing.assert_allclose(r.phat[0], want_ph, rtol=1e-12)
    assert abs(r.expected_len[0] - sum(want_ph)) < 1e-12


def test_n1_is_the_roots_most_probable_token(tab):
    r = _build(tab, [17], 1, 4, 5)
    x, p = _defs.np_row_probs(tab, 17, 0)
    j = int(_defs.np_topk(x, 1)[0])
    assert r.n_sel[0] == 1 and r.token[0, 0] == j and r.parent[0, 0] == -1
    assert abs(r.phat[0, 0] - p[j]) < 1e-12
    assert r.depth_reached[0] == 1                       # depth is capped by n


def test_full_layers_give_d_times_n_drafted_nodes_and_first_layer_min_n_k(tab):
    # first layer holds min(n, k) nodes; with k*|frontier| >= n later layers are full
    r = _build(tab, [1], 8, 3, 4)
    assert r.n_sel[0] == 8
    assert (r.depth[0] == 1).sum() <= 3


def test_threshold_controls_depth(tab):
    deep = _build(tab, range(8), 16, 4, 8, NEG_INF)
    assert np.all(deep.depth_reached == 8)
    for delta in (0.0, 0.2, 0.7, 5.0):
        r = _build(tab, range(8), 16, 4, 8, delta)
        assert np.all(r.depth_reached <= 8) and np.all(r.depth_reached >= 1)
        for b in range(8):
            tr = np.concatenate([[0.0], r.esub_trace[b, :r.depth_reached[b]]])
            gains = np.diff(tr)
            assert np.all(gains[:-1] > delta)                                  # every continued layer cleared delta
            assert r.depth_reached[b] == 8 or not gains[-1] > delta           # the last one did not (or the cap hit)
    assert np.all(_build(tab, range(8), 16, 4, 8, 5.0).depth_reached == 1)


def test_force_depth_overrides_the_threshold(tab):
    r = oracle.table_step(tab, None, np.array([2, 3], np.int32), 16, 4, 8, 0.2,
                          force_depth=np.array([3, 5], np.int32))
    assert r.depth_reached.tolist() == [3, 5]


def test_shared_prefix_is_stored_once():
    # Two 5-token sequences sharing a 3-token prefix need 7 tree nodes, not 10.
    seqs = [(1, 2, 3, 4, 5), (1, 2, 3, 6, 7)]

    def draft(_root, path):
        out = [-20.0] * 8
        nxt = {s[len(path)] for s in seqs if len(s) > len(path) and s[:len(path)] == tuple(path)}
        for t in nxt:
            out[t] = 0.0
        return out

    r = oracle.build_cb(draft, 0, 8, 7, 2, 5, -math.inf)
    got = set(_defs.paths_of(r["token"], r["parent"], r["n_sel"]))
    want = {s[:i] for s in seqs for i in range(1, 6)}
    assert r["n_sel"] == 7 and got == want
