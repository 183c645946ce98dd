"""Helpers for the -m gpu tests: move tables to the device, run one step through the C ABI binding with
poison-filled output buffers, and keep a record of how the comparisons with the oracle came out."""
from __future__ import annotations

import json
import os

import numpy as np
import torch

from paper_2406_17276_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PARITY_LOG = os.path.join(ROOT, "gpurun_out", "parity_counts.json")


def dev_table(tab: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> device tensor (int16 view of the same bytes)."""
    return torch.from_numpy(tab.view(np.int16)).cuda()


def poison(*tensors):
    """Every byte 0xFF: a result the library fails to write shows up as -1 / NaN, never as a stale value."""
    for t in tensors:
        if t is not None:
            t.view(torch.uint8).fill_(0xFF)
    return tensors


def poisoned_tree(ot: binding.OptTree, B: int, trace: bool = True) -> binding.Tree:
    tree = ot.alloc_tree(B, trace=trace)
    poison(tree.token, tree.parent, tree.depth, tree.phat, tree.n_sel, tree.depth_reached, tree.expected_len, tree.esub_trace)
    return tree


def poisoned_verify_out(ot: binding.OptTree, B: int):
    i32 = dict(dtype=torch.int32, device=ot.device)
    D = ot.cfg.max_depth
    return poison(torch.empty(B, **i32), torch.empty((B, D + 1), **i32), torch.empty((B, D), **i32), torch.empty(B, **i32))


def gpu_step(ot: binding.OptTree, d_ld, d_lt, roots: np.ndarray, delta: float, base_pos: np.ndarray | None = None):
    """build + mask + verify into poison-filled buffers; returns a dict of numpy arrays."""
    r = torch.from_numpy(np.ascontiguousarray(roots, np.int32)).cuda()
    B = r.shape[0]
    bp = None if base_pos is None else torch.from_numpy(np.ascontiguousarray(base_pos, np.int32)).cuda()
    tree = ot.build(d_ld, r, delta, poisoned_tree(ot, B))
    mask, pos = poison(torch.empty((B, ot.cfg.n, ot.W), dtype=torch.int64, device=ot.device),
                       torch.empty((B, ot.cfg.n), dtype=torch.int32, device=ot.device))
    ot.mask(tree, bp, mask, pos)
    out = dict(token=tree.token, parent=tree.parent, depth=tree.depth, phat=tree.phat, n_sel=tree.n_sel,
               depth_reached=tree.depth_reached, expected_len=tree.expected_len, esub_trace=tree.esub_trace,
               mask=mask, position_ids=pos)
    if d_lt is not None:
        al, at, an, nr = ot.verify(tree, d_lt, r, poisoned_verify_out(ot, B))
        out.update(accept_len=al, accept_tokens=at, accept_nodes=an, next_root=nr)
    torch.cuda.synchronize()
    assert ot.device_status() == 0
    return {k: v.cpu().numpy() for k, v in out.items()}


def tree_dict(tree: binding.Tree) -> dict:
    return {f: getattr(tree, f).cpu().numpy() for f in
            ("token", "parent", "depth", "phat", "n_sel", "depth_reached", "expected_len", "esub_trace")
            if getattr(tree, f) is not None}


def new_totals() -> dict:
    return dict(exact=0, near_tie=0, stop_near_tie=0, max_phat_rel=0.0, max_elen_rel=0.0)


def add_stats(total: dict, st: dict) -> dict:
    for k in ("exact", "near_tie", "stop_near_tie"):
        total[k] += st[k]
    for k in ("max_phat_rel", "max_elen_rel"):
        total[k] = max(total[k], st[k])
    return total


def record_parity(test_id: str, stats: dict) -> None:
    """Adds one test's comparison counts (sequences that matched the oracle exactly, sequences exempted as
    near-ties of a selection or of the loop test, largest relative errors) to a JSON file next to the other
    run outputs, so that a run leaves a record of how much it leaned on the exemptions."""
    try:
        os.makedirs(os.path.dirname(PARITY_LOG), exist_ok=True)
        rec = json.load(open(PARITY_LOG)) if os.path.exists(PARITY_LOG) else {}
        rec[test_id] = stats
        tot = new_totals()
        for k, v in rec.items():
            if k != "_total":
                add_stats(tot, v)
        rec["_total"] = tot
        with open(PARITY_LOG, "w") as f:
            json.dump(rec, f, indent=1, sort_keys=True)
    except OSError:
        pass
