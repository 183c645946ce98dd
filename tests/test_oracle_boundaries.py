"""Pins for the two oracle outputs that decide which GPU mismatches the parity tests forgive:
min_gap (smallest relative gap at a selection boundary) and stop_margin (smallest distance of a
loop-test gain from the threshold), and for the tie rule of the greedy walk's argmax."""
import json
import math
import os

import numpy as np
import pytest

import oracle
from tests import _defs

G = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_example_eq2_eq3.json")))
V, K = G["V"], G["k"]


def _draft(_root, path):
    key = ",".join(str(t) for t in path)
    return [math.log(x) for x in G["draft_distributions"].get(key, G["default_distribution"])]


@pytest.mark.parametrize("case", G["boundaries_n4"]["cases"])
def test_hand_example_gaps_and_margins(case):
    r = oracle.build_cb(_draft, 0, V, 4, K, case["max_depth"], case["delta"])
    assert r["depth_reached"] == case["depth_reached"]
    if case["min_gap"] is None:              # one layer that keeps every candidate: no boundary, no loop test
        assert r["min_gap"] == math.inf and r["stop_margin"] == math.inf
    else:
        assert r["min_gap"] == pytest.approx(case["min_gap"], rel=1e-12)
        assert r["stop_margin"] == pytest.approx(case["stop_margin"], rel=1e-12)


def test_hand_example_every_boundary_on_its_own():
    """Each boundary of the worked example is isolated by choosing n and the depth so that it is the
    smallest: a gap taken on the wrong pair or at the wrong selection fails one of these."""
    b = G["boundaries_n4"]
    # n = 4, two layers: min(layer-2 gap 1/6, running gap 4/9)
    assert oracle.build_cb(_draft, 0, V, 4, K, 2, -math.inf)["min_gap"] == pytest.approx(b["layer_gap"][1], rel=1e-12)
    # n = 3, one layer: layer 1 keeps .5,.3,.15 and drops .05 -> 2/3 (the running top-n has no boundary yet)
    assert oracle.build_cb(_draft, 0, V, 3, K, 1, -math.inf)["min_gap"] == pytest.approx((0.15 - 0.05) / 0.15, rel=1e-12)
    # n = 1: layer 1 keeps .5 drops .3 (0.4); layer 2 keeps .31 drops .10 (21/31); T: keeps .5 drops .31 (0.38)
    assert oracle.build_cb(_draft, 0, V, 1, K, 1, -math.inf)["min_gap"] == pytest.approx(0.4, rel=1e-12)
    # (Algorithm 1 caps the depth by n, so n = 1 drafts one layer whatever max_depth says)
    assert oracle.build_cb(_draft, 0, V, 1, K, 3, -math.inf)["depth_reached"] == 1
    # n = 2, two layers: layer 1 .3 | .15 -> 0.5; layer 2 .27 | .10 -> 17/27; T {.5,.3,.31,.27}: .31 | .3 -> 1/31
    assert oracle.build_cb(_draft, 0, V, 2, K, 2, -math.inf)["min_gap"] == pytest.approx(0.01 / 0.31, rel=1e-10)
    # the loop test is strict: a gain equal to delta stops, and the margin is zero
    r = oracle.build_cb(_draft, 0, V, 4, K, 3, 1.0)
    assert r["depth_reached"] == 1 and r["stop_margin"] == 0.0


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("n,k,D,delta", [(3, 2, 3, -math.inf), (5, 3, 3, 0.05), (4, 8, 3, 0.3), (6, 2, 4, 0.0), (2, 8, 2, 0.6)])
def test_gaps_and_margins_equal_a_numpy_replay(seed, n, k, D, delta):
    tab = _defs.small_table(32, 8, 100 + seed, peaked=(seed % 2 == 0))
    root = seed % 8
    r = oracle.table_step(tab, None, np.array([root], np.int32), n, k, D, delta)
    gap, margin, d = _defs.beam_boundaries(tab, root, n, k, D, delta)
    assert r.depth_reached[0] == d
    assert r.min_gap[0] == pytest.approx(gap, rel=1e-9) or (math.isinf(gap) and math.isinf(r.min_gap[0]))
    assert r.stop_margin[0] == pytest.approx(margin, rel=1e-9, abs=1e-15) or (math.isinf(margin) and math.isinf(r.stop_margin[0]))


def test_exact_tie_at_a_boundary_has_gap_zero():
    p = [0.4, 0.4, 0.1, 0.1]
    r = oracle.build_cb(lambda _r, _p: [math.log(x) for x in p], 0, 4, 1, 4, 1, -math.inf)
    assert r["min_gap"] == 0.0 and r["token"][0] == 0              # and the tie goes to the lower candidate index


@pytest.mark.parametrize("eps,exempt", [(5e-7, True), (2e-6, False)])
def test_constructed_gap_just_inside_and_outside_the_exemption(eps, exempt):
    p = [0.5, 0.5 * (1.0 - eps), 0.25 * eps, 0.25 * eps]
    r = oracle.build_cb(lambda _r, _p: [math.log(x) for x in p], 0, 4, 1, 4, 1, -math.inf)
    assert r["min_gap"] == pytest.approx(eps, rel=1e-6)
    from tests import _compare
    assert (r["min_gap"] < _compare.GAP_EXEMPT) == exempt


def test_gap_when_the_last_kept_value_is_zero():
    """A kept value of exactly zero can only be followed by dropped values of zero: an exact tie, gap 0
    (0/0 is never formed)."""
    logits = [0.0, -math.inf, -math.inf, -math.inf]
    r = oracle.build_cb(lambda _r, _p: logits, 0, 4, 2, 4, 1, -math.inf)
    assert r["phat"].tolist() == [1.0, 0.0] and r["min_gap"] == 0.0


def test_greedy_walk_takes_the_lowest_token_of_a_tied_target_maximum():
    e = G["n4"]                                   # tokens [0,1,0,0], parents [-1,-1,0,1]

    def target(_root, path):
        if path == ():
            return [5.0, 5.0, 0.0, 0.0]           # tie between tokens 0 and 1 -> 0 (node a), not 1 (node b)
        if path == (0,):
            return [2.0, 1.0, 2.0, 2.0]           # tie between 0, 2, 3 -> 0 (node a0)
        return [0.0, 0.0, 7.0, 7.0]               # tie between 2 and 3 -> 2, no such child: bonus token
    r = oracle.verify_cb(target, 0, V, 4, 3, e["token"], e["parent"], e["depth"])
    assert r["accept_len"] == 3
    assert r["accept_tokens"][:3].tolist() == [0, 0, 2] and r["accept_nodes"][:2].tolist() == [0, 2]
    assert r["next_root"] == 2
