"""Helpers for the -m gpu tests: move tables to the device and run one step through the C ABI binding."""
from __future__ import annotations

import numpy as np
import torch

from paper_2406_17276_b200 import binding


def dev_table(tab: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> device tensor (int16 view of the same bytes)."""
    return torch.from_numpy(tab.view(np.int16)).cuda()


def gpu_step(ot: binding.OptTree, d_ld, d_lt, roots: np.ndarray, delta: float, base_pos: np.ndarray | None = None):
    """build + mask + verify; returns a dict of numpy arrays."""
    r = torch.from_numpy(np.ascontiguousarray(roots, np.int32)).cuda()
    bp = None if base_pos is None else torch.from_numpy(np.ascontiguousarray(base_pos, np.int32)).cuda()
    tree = ot.build(d_ld, r, delta)
    mask, pos = ot.mask(tree, bp)
    out = dict(token=tree.token, parent=tree.parent, depth=tree.depth, phat=tree.phat, n_sel=tree.n_sel,
               depth_reached=tree.depth_reached, expected_len=tree.expected_len, esub_trace=tree.esub_trace,
               mask=mask, position_ids=pos)
    if d_lt is not None:
        al, at, an, nr = ot.verify(tree, d_lt, r)
        out.update(accept_len=al, accept_tokens=at, accept_nodes=an, next_root=nr)
    torch.cuda.synchronize()
    assert ot.device_status() == 0
    return {k: v.cpu().numpy() for k, v in out.items()}
