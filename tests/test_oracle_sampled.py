"""Pins of the oracle's verification with sampling: the generator, the inverse-CDF draw, the walk."""
import math

import numpy as np

import oracle
from paper_2406_17276_b200 import synth


def test_philox_known_answers():
    """Known-answer vectors of Philox4x32-10 as published with the generator (Random123's kat_vectors)."""
    z = oracle.philox4x32_10([0, 0, 0, 0], [0, 0])
    assert [int(v) for v in z] == [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]
    f = oracle.philox4x32_10([0xFFFFFFFF] * 4, [0xFFFFFFFF] * 2)
    assert [int(v) for v in f] == [0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD]
    p = oracle.philox4x32_10([0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344], [0xA4093822, 0x299F31D0])
    assert [int(v) for v in p] == [0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1]


def test_philox_is_a_bijection_on_a_small_cube():
    """Independent of the constants: for a fixed key the block function never maps two counters to one output."""
    seen = set()
    for a in range(64):
        for b in range(16):
            seen.add(tuple(int(v) for v in oracle.philox4x32_10([a, b, 0, 0], [7, 9])))
    assert len(seen) == 64 * 16


def test_uniforms_are_uniform():
    u = np.array([oracle.uniform(12345, 3, b, j) for b in range(40) for j in range(250)])
    assert (u >= 0).all() and (u < 1).all()
    hist, _ = np.histogram(u, bins=20, range=(0, 1))
    assert hist.min() > 380 and hist.max() < 620                                   # 500 expected per bin
    assert abs(u.mean() - 0.5) < 0.01 and len(np.unique(u)) == u.size
    assert oracle.uniform(1, 0, 0, 0) != oracle.uniform(2, 0, 0, 0) != oracle.uniform(1, 1, 0, 0)


def test_draw_is_the_inverse_cdf():
    """numpy's cumulative sum and searchsorted are the independent definition."""
    rng = np.random.default_rng(0)
    for tau in (0.3, 1.0, 2.5):
        x = rng.normal(0, 3, 300)
        e = np.exp((x - x.max()) / tau); cdf = np.cumsum(e)
        for u in list(rng.random(200)) + [0.0, 0.999999999]:
            y, margin = oracle.sample_token(x, tau, u)
            want = int(np.searchsorted(cdf, u * cdf[-1], side="right"))
            assert y == min(want, 299) or margin < 1e-12
    # frequencies follow softmax(x / tau)
    x = np.array([2.0, 1.0, 0.0, -1.0]); tau = 0.7
    p = np.exp(x / tau); p /= p.sum()
    us = (np.arange(20000) + 0.5) / 20000
    counts = np.bincount([oracle.sample_token(x, tau, u)[0] for u in us], minlength=4)
    assert np.abs(counts / 20000 - p).max() < 2e-4


def test_special_rows():
    x = np.full(50, -np.inf); x[17] = 3.0
    assert all(oracle.sample_token(x, 1.0, u)[0] == 17 for u in (0.0, 0.3, 0.99999))          # one finite logit
    x = np.zeros(10)
    assert [oracle.sample_token(x, 1.0, (i + 0.5) / 10)[0] for i in range(10)] == list(range(10))   # constant row: uniform
    x = np.array([0.0, 5.0, 1.0])
    assert all(oracle.sample_token(x, 1e-3, u)[0] == 1 for u in (0.0, 0.5, 0.999))              # tau -> 0: the argmax


def test_walk_follows_the_sampled_tokens():
    w = synth.Workload("sv", 8, 512, 24, 5, 7, 3.0, 1.1, 0.3, H=64, seed=4)
    ld, lt = synth.make_tables(w)
    roots = synth.root_tokens(w.batch, w.V, 2)
    r = oracle.table_step(ld, lt, roots, w.n, w.k, w.max_depth, -math.inf)
    lt_f = synth.bf16_bits_to_f32(lt).astype(np.float64)
    for tau, seed, step in ((1.0, 7, 0), (0.5, 7, 1), (1e-4, 9, 0)):
        s = oracle.table_verify_sampled(lt, roots, r.token, r.parent, r.depth, r.n_sel, w.max_depth, tau, seed, step)
        for b in range(w.batch):
            A = int(s["accept_len"][b])
            assert 1 <= A <= int(r.depth_reached[b]) + 1 and s["next_root"][b] == s["accept_tokens"][b, A - 1]
            cur, dep = -1, 0
            for j in range(A):                                   # replay the walk with the definition's pieces
                tok_path = []
                a = cur
                while a >= 0:
                    tok_path.append(int(r.token[b, a])); a = int(r.parent[b, a])
                t_here = roots[b] if cur < 0 else int(r.token[b, cur])
                row = (t_here * 31 + dep) % ld.shape[0]
                y, _ = oracle.sample_token(lt_f[row], tau, oracle.uniform(seed, step, b, cur + 1))
                assert s["accept_tokens"][b, j] == y
                kids = [i for i in range(int(r.n_sel[b])) if r.parent[b, i] == cur and r.token[b, i] == y]
                if j < A - 1:
                    assert kids == [int(s["accept_nodes"][b, j])]
                    cur = kids[0]; dep = int(r.depth[b, cur])
                else:
                    assert kids == []
        if tau < 1e-3:                                           # nearly greedy: the greedy walk's result
            assert np.array_equal(s["accept_len"], r.accept_len) and np.array_equal(s["accept_tokens"], r.accept_tokens)
