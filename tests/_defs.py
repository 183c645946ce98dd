"""Plain NumPy restatements of the definitions the oracle is pinned against.

Nothing here calls the oracle or the CUDA library: it is the "something other
than itself" the oracle is checked with (softmax / ranking by library routines,
exhaustive enumeration, path enumeration).
"""
from __future__ import annotations

import itertools

import numpy as np

from paper_2406_17276_b200 import synth


def small_table(H, V, seed, sigma=3.0, peaked=True):
    """A small bf16 table with the same recipe as the full-size ones."""
    if peaked:
        return synth.draft_table(V, sigma, 1.1, seed, H=H, rows_per_block=64)
    rng = np.random.default_rng(seed)
    return synth.f32_to_bf16_bits((sigma * rng.standard_normal((H, V))).astype(np.float32))


def row_index(token, depth, H):
    return (int(token) * 31 + int(depth)) % H


def np_row_probs(table, token, depth):
    """fp64 softmax of the row a (token, depth) node reads, by NumPy."""
    H = table.shape[0]
    x = synth.bf16_bits_to_f32(table[row_index(token, depth, H)]).astype(np.float64)
    e = np.exp(x - x.max())
    return x, e / e.sum()


def np_topk(x, k):
    """Indices of the k largest entries ranked (value desc, index asc) via lexsort."""
    order = np.lexsort((np.arange(x.shape[0]), -x))
    return order[:k]


def full_tree(table, root_token, k, D):
    """All nodes of the k-restricted draft tree down to depth D.

    Returns a list of (path_tuple, phat, parent_index) in breadth-first order
    (a parent always precedes its children); parent_index -1 = child of the root.
    """
    nodes = []
    frontier = [((), 1.0, -1, root_token, 0)]   # (path, phat, index, token, depth)
    for d in range(1, D + 1):
        nxt = []
        for path, ph, idx, tok, dep in frontier:
            x, p = np_row_probs(table, tok, dep)
            for j in np_topk(x, min(k, x.shape[0])):
                nodes.append((path + (int(j),), ph * p[j], idx))
                nxt.append((path + (int(j),), ph * p[j], len(nodes) - 1, int(j), d))
        frontier = nxt
    return nodes


def best_closed_subset(nodes, n):
    """Exhaustive maximum of sum(phat) over parent-closed subsets of exactly min(n, len) nodes.

    Nodes are in an order where parents precede children, so every closed set is
    generated exactly once as an increasing index sequence whose every element's
    parent is already present.
    """
    N = len(nodes)
    n = min(n, N)
    best = [-1.0, None]
    ph = [nd[1] for nd in nodes]
    par = [nd[2] for nd in nodes]

    def rec(start, chosen, inset, total):
        if len(chosen) == n:
            if total > best[0]:
                best[0], best[1] = total, tuple(chosen)
            return
        for i in range(start, N):
            if par[i] == -1 or par[i] in inset:
                chosen.append(i); inset.add(i)
                rec(i + 1, chosen, inset, total + ph[i])
                chosen.pop(); inset.discard(i)

    rec(0, [], set(), 0.0)
    return best[0], {nodes[i][0] for i in best[1]}


def best_closed_subset_literal(nodes, n):
    """Same maximum by testing every size-n subset of the node set (tiny cases only)."""
    N = len(nodes)
    n = min(n, N)
    best, best_set = -1.0, None
    for comb in itertools.combinations(range(N), n):
        s = set(comb)
        if all(nodes[i][2] == -1 or nodes[i][2] in s for i in comb):
            tot = sum(nodes[i][1] for i in comb)
            if tot > best:
                best, best_set = tot, {nodes[i][0] for i in comb}
    return best, best_set


def paths_of(token, parent, n_sel):
    """Root-to-node token paths of a packed tree."""
    out = []
    for i in range(n_sel):
        p, a = [], i
        while a >= 0:
            p.append(int(token[a])); a = int(parent[a])
        out.append(tuple(reversed(p)))
    return out


def target_chain(table, root_token, length):
    """The target's greedy continuation: token after the root, after that token, ..."""
    chain, tok, dep = [], root_token, 0
    for _ in range(length):
        x, _p = np_row_probs(table, tok, dep)
        y = int(np_topk(x, 1)[0])
        chain.append(y)
        tok, dep = y, dep + 1
    return chain


def beam_boundaries(table, root_token, n, k, D, delta):
    """The boundaries Algorithm 1 decides at, replayed with NumPy sorts on the nodes of full_tree.

    Per drafted layer: the relative gap (kept - dropped) / kept between the last candidate that
    enters the layer and the best one that does not, the same gap for the n largest nodes of T,
    and |gain - delta| of every loop test that is evaluated.  Returns (smallest gap or inf,
    smallest margin or inf, layers drafted).
    """
    D = min(D, n)
    nodes = full_tree(table, root_token, k, D)            # (path, phat, parent index), breadth first
    kids = {}
    for i, (path, ph, par) in enumerate(nodes):
        kids.setdefault(par, []).append(i)                # in sibling-rank order
    gap, margin, E, T, layer = np.inf, np.inf, 0.0, [], [-1]
    d = 0
    while True:
        d += 1
        cand = [c for f in layer for c in kids.get(f, [])]          # candidate-index order
        ph = np.array([nodes[c][1] for c in cand])
        order = np.lexsort((np.arange(len(cand)), -ph))
        nl = min(n, len(cand))
        if len(cand) > nl:
            gap = min(gap, (ph[order[nl - 1]] - ph[order[nl]]) / ph[order[nl - 1]])
        layer = [cand[i] for i in sorted(order[:nl])]
        T += layer
        tp = np.sort(np.array([nodes[i][1] for i in T]))[::-1]
        nR = min(n, len(T))
        if len(T) > nR:
            gap = min(gap, (tp[nR - 1] - tp[nR]) / tp[nR - 1])
        esub = float(tp[:nR].sum())
        if d >= D:
            break
        margin = min(margin, abs((esub - E) - delta))
        if not (esub - E > delta):
            break
        E = esub
    return gap, margin, d
