"""Pins: tree attention mask / position ids by definition, and greedy verification by path enumeration."""
import numpy as np
import pytest

import oracle
from paper_2406_17276_b200 import synth
from tests import _defs

NEG_INF = float("-inf")


@pytest.mark.parametrize("n,k,D", [(10, 10, 6), (64, 10, 10), (100, 8, 12), (256, 32, 20), (512, 16, 10), (1000, 32, 8)])
def test_mask_is_ancestor_or_self_by_parent_walk(n, k, D):
    tab = _defs.small_table(128, 1024, 31)
    base = np.array([7, 1000], np.int32)
    r = oracle.table_step(tab, None, np.array([4, 9], np.int32), n, k, D, NEG_INF, base_pos=base)
    W = (n + 63) // 64
    assert r.mask.shape == (2, n, W)
    for b in range(2):
        ns = int(r.n_sel[b])
        for i in range(n):
            bits = {j for j in range(n) if (int(r.mask[b, i, j // 64]) >> (j % 64)) & 1}
            if i >= ns:
                assert bits == set() and r.position_ids[b, i] == 0
                continue
            anc, a = set(), i
            while a >= 0:
                anc.add(a); a = int(r.parent[b, a])
            assert bits == anc
            assert len(bits) == r.depth[b, i]                       # popcount = depth
            assert r.position_ids[b, i] == base[b] + r.depth[b, i]   # a layer shares one position index


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_verify_equals_longest_branch_following_the_target_chain(seed):
    w = synth.Workload("t", 8, 512, 24, 6, 8, 3.0, 1.1, 0.30, H=256, seed=seed)
    ld, lt = synth.make_tables(w)
    roots = synth.root_tokens(8, w.V, seed)
    r = oracle.table_step(ld, lt, roots, w.n, w.k, w.max_depth, NEG_INF)
    lens = []
    for b in range(8):
        chain = _defs.target_chain(lt, int(roots[b]), w.max_depth + 1)
        paths = _defs.paths_of(r.token[b], r.parent[b], r.n_sel[b])
        hits = max([len(p) for p in paths if tuple(chain[:len(p)]) == p] + [0])
        A = hits + 1
        assert r.accept_len[b] == A
        assert 1 <= A <= r.depth_reached[b] + 1
        assert r.accept_tokens[b, :A].tolist() == chain[:A]
        assert np.all(r.accept_tokens[b, A:] == -1)
        assert r.next_root[b] == chain[A - 1]
        for j in range(A - 1):
            assert paths[r.accept_nodes[b, j]] == tuple(chain[:j + 1])
        assert np.all(r.accept_nodes[b, A - 1:] == -1)
        lens.append(A)
    assert len(set(lens)) > 1 or lens[0] > 1       # the workload actually exercises acceptance


def test_identical_draft_and_target_accept_the_greedy_chain():
    tab = _defs.small_table(256, 512, 5)
    roots = np.arange(6, dtype=np.int32) * 13
    r = oracle.table_step(tab, tab, roots, 24, 6, 8, NEG_INF)
    for b in range(6):
        chain = _defs.target_chain(tab, int(roots[b]), 9)
        paths = set(_defs.paths_of(r.token[b], r.parent[b], r.n_sel[b]))
        L = 0
        while L < 8 and tuple(chain[:L + 1]) in paths:
            L += 1
        assert r.accept_len[b] == L + 1 >= 2       # the draft's top token is always in the tree


def test_target_that_never_matches_accepts_only_the_bonus_token():
    V = 64
    ld = _defs.small_table(64, V, 8)
    lt = ld.copy()
    lt[:, :] = synth.f32_to_bf16_bits(np.float32(-30.0))
    # the target always answers with token V-1, which the draft never proposes (make it very unlikely)
    ld[:, V - 1] = synth.f32_to_bf16_bits(np.float32(-60.0))
    lt[:, V - 1] = synth.f32_to_bf16_bits(np.float32(9.0))
    r = oracle.table_step(ld, lt, np.array([1, 2, 3], np.int32), 8, 4, 4, NEG_INF)
    assert r.accept_len.tolist() == [1, 1, 1]
    assert r.next_root.tolist() == [V - 1] * 3
