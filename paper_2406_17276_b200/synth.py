"""Seeded synthetic inputs: bf16 logit tables and root tokens.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no softmax, no top-k, no tree logic), so that the
CUDA path and the CPU oracle can both be fed the very same bytes without
sharing any code that could hide a common mistake.

The synthetic draft and target "models" are logit tables of shape [H, V] in
bf16 (stored as uint16 bit patterns).  A child of token ``t`` at depth ``d``
reads row ``(t*31 + d) mod H``; that addressing rule lives in the consumers,
not here.

Recipe for one table row ``r``:
  * every entry is ``sigma * N(0, 1)`` (float32 draws),
  * one "peak" token ``c_r`` (uniform over the vocabulary) gets a bias
    ``b_r = ln V + sigma^2/2 + b0 - ln z_r`` added, where ``z_r`` is drawn from a
    Zipf(s) law truncated to ``{1..1024}``.  ``ln V + sigma^2/2`` is the log of the
    expected background mass ``V * E[exp(sigma*N)]``, so the peak's odds against
    the background are about ``exp(b0)/z_r``: rank 1 gives a ~0.98 peak, rank
    100 a ~0.35 peak.
  * the result is rounded to bf16 (round to nearest even).

The target table is a copy of the draft table in which, on a seeded subset
of exactly ``round(q*H)`` rows, the row's largest element is swapped with the
element at another seeded position holding a strictly smaller value, so the
draft and target argmaxes disagree on exactly that fraction of rows and the
row statistics are unchanged.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

H_ROWS = 4096          # rows in every synthetic table
ROW_MUL = 31           # row = (token*ROW_MUL + depth) mod H, applied by the consumers
ZIPF_TRUNC = 1024      # the Zipf rank is truncated to 1..ZIPF_TRUNC
PEAK_B0 = 4.0          # log-odds of a rank-1 peak against the Gaussian background


@dataclasses.dataclass(frozen=True)
class Workload:
    """One measurement / parity configuration."""
    name: str
    batch: int
    V: int
    n: int
    k: int
    max_depth: int
    sigma: float
    zipf_s: float
    disagree: float      # fraction of rows whose draft/target argmaxes differ
    H: int = H_ROWS
    seed: int = 2406_17276


# The five configurations the build is measured / checked on.
WORKLOADS = {
    "c1": Workload("c1", 1, 32000, 10, 10, 6, 3.0, 1.1, 0.20),
    "c2": Workload("c2", 1, 32000, 50, 10, 10, 4.0, 1.3, 0.10),
    "c3": Workload("c3", 1, 128256, 64, 16, 12, 3.0, 1.1, 0.20),
    "c4": Workload("c4", 32, 32000, 64, 10, 10, 3.0, 1.1, 0.20),
    "c5": Workload("c5", 64, 152064, 256, 32, 20, 2.5, 1.05, 0.20),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _zipf_ranks(u: np.ndarray, s: float, trunc: int = ZIPF_TRUNC) -> np.ndarray:
    """Inverse-CDF draw from Zipf(s) truncated to 1..trunc, from uniforms u in [0,1)."""
    w = np.arange(1, trunc + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    return np.minimum(np.searchsorted(cdf, u, side="right"), trunc - 1) + 1


def draft_table(V: int, sigma: float, zipf_s: float, seed: int, H: int = H_ROWS,
                rows_per_block: int = 256) -> np.ndarray:
    """The draft logit table L_d: uint16 [H, V] of bf16 bit patterns."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x4C64]))
    peak_tok = rng.integers(0, V, size=H, dtype=np.int64)
    ranks = _zipf_ranks(rng.random(H), zipf_s)
    bias = (math.log(V) + 0.5 * sigma * sigma + PEAK_B0 - np.log(ranks.astype(np.float64))).astype(np.float32)
    out = np.empty((H, V), dtype=np.uint16)
    for r0 in range(0, H, rows_per_block):
        r1 = min(H, r0 + rows_per_block)
        blk = rng.standard_normal((r1 - r0, V), dtype=np.float32)
        blk *= np.float32(sigma)
        rr = np.arange(r1 - r0)
        blk[rr, peak_tok[r0:r1]] += bias[r0:r1]
        out[r0:r1] = f32_to_bf16_bits(blk)
    return out


def target_table(draft: np.ndarray, disagree: float, seed: int) -> np.ndarray:
    """The target logit table L_t derived from L_d (see the module docstring)."""
    H, V = draft.shape
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x4C74]))
    out = draft.copy()
    n_swap = int(round(disagree * H))
    rows = rng.permutation(H)[:n_swap]
    for r in rows:
        vals = bf16_bits_to_f32(out[r])
        i = int(np.argmax(vals))
        j = int(rng.integers(0, V))
        tries = 0
        while not (vals[j] < vals[i]):      # needs a strictly smaller partner
            j = (j + 1) % V
            tries += 1
            if tries > V:                   # constant row: nothing to swap
                break
        out[r, i], out[r, j] = out[r, j], out[r, i]
    return out


def root_tokens(batch: int, V: int, seed: int) -> np.ndarray:
    """First root token of every sequence: int32 [batch]."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x526F]))
    return rng.integers(0, V, size=batch, dtype=np.int64).astype(np.int32)


def make_tables(w: Workload, H: int | None = None, V: int | None = None):
    """(L_d, L_t) for a workload; H / V can be overridden to build reduced cases."""
    H = w.H if H is None else H
    V = w.V if V is None else V
    ld = draft_table(V, w.sigma, w.zipf_s, w.seed, H)
    lt = target_table(ld, w.disagree, w.seed)
    return ld, lt
