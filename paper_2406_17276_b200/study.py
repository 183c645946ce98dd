"""Acceptance-length study on the synthetic tables (`bench.py --study mal`).

What the paper's experiments ask of the method, minus the real models: does the adaptive tree
accept more tokens per step than a fixed tree of the same size (Tables 1-2: binary tree, sequence
draft), how does the acceptance length grow with the node budget (Section 4.3), and does E(A)
track the acceptance length A that verification then finds (Section 4.2's joint histogram).

Everything the library computes goes through its C ABI (opt_tree_build, opt_tree_verify,
opt_tree_row_softmax_topk).  The fixed-shape trees are the comparison, not the method: they are
assembled here from the row step's top tokens (a complete b-ary tree cut off at n nodes, level by
level; the sequence draft is the chain of most probable tokens, which is opt_tree_build with
k = 1) and verified by the same opt_tree_verify.  Every shape is tried on the same root tokens.
Every step draws fresh seeded root tokens: the table model's whole state is the root token, so a
chain that feeds on its own accepted tokens (Algorithm 2's Concat) falls into a cycle of a few dozen
roots within a few steps and would sample nothing else (the parity tests follow such chains; a
study of averages must not).  The adaptive tree is built twice: with the workload's depth limit,
and with Algorithm 1's own limit (depth < n; here min(n, 500) layers) and threshold 0, which is
the setting in which no tree of n nodes from the same candidates can have a larger E(A).
"""
from __future__ import annotations

import math
import time

import numpy as np

from . import synth

NEG_INF = -math.inf


def _bary_tree(ot, d_ld, roots, b, n, H):
    """Complete b-ary tree of n nodes under every root, packed level by level (parents before children,
    siblings by rank).  Returns a binding.Tree with path values (Eq. 2) and E(A) (Eq. 3)."""
    import torch
    from .binding import Tree
    B = roots.shape[0]
    dev = roots.device
    tok = torch.full((B, n), -1, dtype=torch.int32, device=dev)
    par = torch.full((B, n), -1, dtype=torch.int32, device=dev)
    dep = torch.zeros((B, n), dtype=torch.int32, device=dev)
    ph = torch.zeros((B, n), dtype=torch.float64, device=dev)
    f_tok = roots.view(B, 1).to(torch.int64)
    f_ph = torch.ones((B, 1), dtype=torch.float64, device=dev)
    f_idx = torch.full((1,), -1, dtype=torch.int64, device=dev)        # packed index of each frontier node
    filled, level = 0, 0
    while filled < n:
        level += 1
        F = f_tok.shape[1]
        rows = ((f_tok * 31 + (level - 1)) % H).to(torch.int32).reshape(-1)
        tk, pr = ot.row_softmax_topk(d_ld, rows)                       # [B*F, k]
        take = min(F * b, n - filled)
        c_tok = tk[:, :b].reshape(B, F * b)[:, :take]
        c_ph = (f_ph.unsqueeze(2) * pr[:, :b].reshape(B, F, b)).reshape(B, F * b)[:, :take]
        c_par = f_idx.repeat_interleave(b)[:take]
        tok[:, filled:filled + take] = c_tok
        par[:, filled:filled + take] = c_par.to(torch.int32)
        dep[:, filled:filled + take] = level
        ph[:, filled:filled + take] = c_ph
        f_tok, f_ph = c_tok.to(torch.int64), c_ph
        f_idx = torch.arange(filled, filled + take, device=dev)
        filled += take
    n_sel = torch.full((B,), n, dtype=torch.int32, device=dev)
    return Tree(tok, par, dep, ph, n_sel, torch.full((B,), level, dtype=torch.int32, device=dev), ph.sum(1), None), level


def run(name: str, steps: int, local: int = 0, n: int | None = None, delta: float = NEG_INF, keep_first: int = 0):
    """`steps` decoding steps on workload `name` (node budget n, default the workload's), each from fresh
    seeded roots: acceptance length and E(A) of the adaptive tree (the workload's depth limit; and depth
    limited by n alone with threshold 0), of the sequence draft and of the binary and 4-ary trees with the
    same number of nodes, on the same roots.  keep_first: the roots of that many first steps are returned
    too (for a check on the host)."""
    import torch
    from . import binding
    w = synth.WORKLOADS[name]
    n = n or w.n
    ld, lt = synth.make_tables(w)
    d_ld = torch.from_numpy(ld.view(np.int16)).cuda()
    d_lt = torch.from_numpy(lt.view(np.int16)).cuda()
    B, D = w.batch, w.max_depth
    dev = f"cuda:{local}"
    ot = binding.OptTree(w.V, w.H, n, w.k, D, B, device=dev)
    Dseq = min(n, 500)
    seq = binding.OptTree(w.V, w.H, n, 1, Dseq, B, device=dev)          # k = 1: the chain of most probable tokens
    deep = binding.OptTree(w.V, w.H, n, w.k, Dseq, B, device=dev)       # Algorithm 1's own depth limit
    tree, chain, dtree = ot.alloc_tree(B, trace=False), seq.alloc_tree(B, trace=False), deep.alloc_tree(B, trace=False)
    shapes = ["opt_tree", "opt_tree_depth_n", "sequence", "binary", "4-ary"]
    A = {s: torch.zeros((steps, B), dtype=torch.int32, device="cuda") for s in shapes}
    E = {s: torch.zeros((steps, B), dtype=torch.float64, device="cuda") for s in shapes}
    depth_of = {}
    kept_roots = []
    i32 = dict(dtype=torch.int32, device="cuda")
    vo = (torch.empty(B, **i32), torch.empty((B, D + 1), **i32), torch.empty((B, D), **i32), torch.empty(B, **i32))
    vs = (torch.empty(B, **i32), torch.empty((B, Dseq + 1), **i32), torch.empty((B, Dseq), **i32), torch.empty(B, **i32))
    t0 = time.perf_counter()
    for s in range(steps):
        roots_np = synth.root_tokens(B, w.V, w.seed + 1 + s)
        roots = torch.from_numpy(roots_np).cuda()
        if s < keep_first:
            kept_roots.append(roots_np.copy())
        ot.build(d_ld, roots, delta, tree)
        ot.verify(tree, d_lt, roots, vo)
        A["opt_tree"][s] = vo[0]; E["opt_tree"][s] = tree.expected_len
        deep.build(d_ld, roots, 0.0, dtree)
        deep.verify(dtree, d_lt, roots, vs)
        A["opt_tree_depth_n"][s] = vs[0]; E["opt_tree_depth_n"][s] = dtree.expected_len
        seq.build(d_ld, roots, NEG_INF, chain)
        seq.verify(chain, d_lt, roots, vs)
        A["sequence"][s] = vs[0]; E["sequence"][s] = chain.expected_len
        for shape, b in (("binary", 2), ("4-ary", 4)):
            ft, lv = _bary_tree(ot, d_ld, roots, b, n, w.H)
            depth_of[shape] = lv
            fv = ot.verify(ft, d_lt, roots) if lv <= D else seq.verify(ft, d_lt, roots)
            A[shape][s] = fv[0]; E[shape][s] = ft.expected_len
    torch.cuda.synchronize()
    if ot.device_status() != 0 or seq.device_status() != 0 or deep.device_status() != 0:
        raise RuntimeError("device status after the study")
    dt = time.perf_counter() - t0
    out = {"workload": f"{name}: batch {B}, V={w.V}, n={n}, k={w.k}, max_depth={D}, delta={'off' if delta == NEG_INF else delta}",
           "steps": steps, "trees_per_shape": steps * B, "seconds": dt, "shapes": {}}
    for s in shapes:
        a, e = A[s].double().cpu().numpy().ravel(), E[s].cpu().numpy().ravel()
        out["shapes"][s] = {"mean_acceptance_length": float(a.mean()), "mean_expected_length_plus_1": float(e.mean() + 1.0),
                            "corr_EA_A": float(np.corrcoef(a, e)[0, 1]) if a.std() > 0 and e.std() > 0 else None}
    out["shapes"]["sequence"]["depth"] = Dseq
    out["shapes"]["opt_tree"]["depth_limit"] = D
    out["shapes"]["opt_tree_depth_n"]["depth_limit"] = Dseq
    for s, lv in depth_of.items():
        out["shapes"][s]["depth"] = lv
    a, e = A["opt_tree"].cpu().numpy().ravel(), E["opt_tree"].cpu().numpy().ravel()
    top = int(max(a.max(), np.rint(e + 1.0).max()))
    hist = np.zeros((top + 1, top + 1), np.int64)
    np.add.at(hist, (np.rint(e + 1.0).astype(np.int64), a.astype(np.int64)), 1)
    out["hist_rows_rounded_EA_plus_1_cols_A"] = hist.tolist()
    first = {"roots": kept_roots, "A": A["opt_tree"][:keep_first].cpu().numpy(), "E": E["opt_tree"][:keep_first].cpu().numpy(),
             "tables": (ld, lt), "w": w, "n": n,
             "A_shapes": {s: A[s][:keep_first].cpu().numpy() for s in shapes},
             "E_shapes": {s: E[s][:keep_first].cpu().numpy() for s in shapes}}
    return out, first
