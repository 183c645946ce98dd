"""Pin: hand-computed example of Eq. 2 / Eq. 3 / Algorithm 1 / Algorithm 2 (tests/golden)."""
import json
import math
import os

import numpy as np
import pytest

import oracle

G = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_example_eq2_eq3.json")))
V, K = G["V"], G["k"]


def _draft(_root, path):
    key = ",".join(str(t) for t in path)
    p = G["draft_distributions"].get(key, G["default_distribution"])
    return [math.log(x) for x in p]


def test_n4_tree_mask_and_esub_trace():
    e = G["n4"]
    r = oracle.build_cb(_draft, 0, V, 4, K, 3, 0.1)
    assert r["n_sel"] == 4 and r["depth_reached"] == e["depth_reached_delta_0p1"]
    assert r["token"].tolist() == e["token"]
    assert r["parent"].tolist() == e["parent"]
    assert r["depth"].tolist() == e["depth"]
    np.testing.assert_allclose(r["phat"], e["phat"], rtol=1e-12)
    np.testing.assert_allclose(r["esub_trace"], e["esub_after_layer"], rtol=1e-12)
    assert abs(r["expected_len"] - e["expected_len"]) < 1e-12
    mask, pos = oracle.mask_of(r["parent"], r["depth"], 4, 4, base_pos=100)
    assert mask[:, 0].tolist() == e["mask"]
    assert pos.tolist() == [101, 101, 102, 102]


def test_threshold_stops_one_layer_earlier_with_same_tree():
    e = G["n4"]
    r = oracle.build_cb(_draft, 0, V, 4, K, 3, 0.5)
    assert r["depth_reached"] == e["depth_reached_delta_0p5"]
    assert r["token"].tolist() == e["token"] and r["parent"].tolist() == e["parent"]
    assert abs(r["expected_len"] - e["expected_len"]) < 1e-12


def test_n5_third_layer_node_replaces_a_first_layer_node():
    e = G["n5"]
    r = oracle.build_cb(_draft, 0, V, 5, K, 3, -math.inf)
    np.testing.assert_allclose(r["esub_trace"], e["esub_after_layer"], rtol=1e-12)
    assert abs(r["expected_len"] - e["expected_len_three_layers"]) < 1e-12
    np.testing.assert_allclose(sorted(r["phat"], reverse=True), e["phat_sorted_desc"], rtol=1e-12)
    assert r["depth"].tolist() == [1, 1, 2, 2, 3]


@pytest.mark.parametrize("case", G["verify_n4"])
def test_greedy_verify_on_the_n4_tree(case):
    e = G["n4"]

    def target(_root, path):
        key = ",".join(str(t) for t in path)
        out = [0.0] * V
        out[case["target_argmax"].get(key, 3)] = 5.0
        return out

    r = oracle.verify_cb(target, 0, V, 4, 3, e["token"], e["parent"], e["depth"])
    A = case["accept_len"]
    assert r["accept_len"] == A
    assert r["accept_tokens"][:A].tolist() == case["accept_tokens"]
    assert r["accept_nodes"][:A - 1].tolist() == case["accept_nodes"]
    assert r["next_root"] == case["accept_tokens"][-1]
