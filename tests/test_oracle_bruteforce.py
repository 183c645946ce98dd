"""Pin: the oracle's tree maximises E(A) (Eq. 3) among all root-containing subtrees.

Exhaustive search over every parent-closed node subset of the k-restricted draft
tree on tiny vocabularies; the search and the probabilities are NumPy/Python and
never call the oracle.
"""
import numpy as np
import pytest

import oracle
from tests import _defs

NEG_INF = float("-inf")


def _oracle_tree(tab, root, n, k, D):
    r = oracle.table_step(tab, None, np.array([root], np.int32), n, k, D, NEG_INF)
    ns = int(r.n_sel[0])
    return r, set(_defs.paths_of(r.token[0], r.parent[0], ns))


@pytest.mark.parametrize("n,k,D", [(1, 8, 2), (3, 8, 2), (4, 8, 2), (5, 8, 3), (6, 2, 3), (6, 3, 3), (4, 2, 4)])
@pytest.mark.parametrize("seed", [11, 12, 13])
def test_oracle_equals_exhaustive_optimum(n, k, D, seed):
    V, H = 8, 64
    tab = _defs.small_table(H, V, seed, sigma=1.0, peaked=False)
    root = seed % V
    nodes = _defs.full_tree(tab, root, k, min(D, n))
    want_val, want_set = _defs.best_closed_subset(nodes, n)
    r, got_set = _oracle_tree(tab, root, n, k, D)
    assert abs(r.expected_len[0] - want_val) < 1e-12
    assert got_set == want_set


@pytest.mark.parametrize("n,k,D", [(4, 2, 3), (6, 2, 3), (3, 3, 2), (4, 8, 1)])
def test_oracle_equals_literal_all_subsets(n, k, D):
    V, H = 8, 64
    tab = _defs.small_table(H, V, 21, sigma=1.0, peaked=False)
    nodes = _defs.full_tree(tab, 5, k, min(D, n))
    want_val, want_set = _defs.best_closed_subset_literal(nodes, n)
    r, got_set = _oracle_tree(tab, 5, n, k, D)
    assert abs(r.expected_len[0] - want_val) < 1e-12
    assert got_set == want_set


def test_two_enumerations_agree():
    tab = _defs.small_table(64, 8, 5, sigma=1.0, peaked=False)
    nodes = _defs.full_tree(tab, 1, 2, 3)
    a = _defs.best_closed_subset(nodes, 5)
    b = _defs.best_closed_subset_literal(nodes, 5)
    assert abs(a[0] - b[0]) < 1e-15 and a[1] == b[1]
