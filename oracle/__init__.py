"""ctypes front end of the CPU oracle (oracle/opt_tree_oracle.c).

TEST INFRASTRUCTURE: only tests, the smoke check and the benchmark's
cpu_baseline / reference legs may import this package.  It never touches the
CUDA library, and the CUDA library never touches it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "opt_tree_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C11, -O2, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"])
    return _LIB


LOGITS_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_double))

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ot_memo_create.restype = C.c_void_p
        _lib.ot_memo_create.argtypes = [C.c_int64, C.c_int32]
        _lib.ot_memo_destroy.argtypes = [C.c_void_p]
        _lib.ot_table_step.restype = C.c_int
        _lib.ot_build_cb.restype = C.c_int
        _lib.ot_verify_cb.restype = C.c_int32
        _lib.ot_row_softmax_topk_bf16.restype = C.c_int32
        _lib.ot_row_argmax_bf16.restype = C.c_int32
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


@dataclass
class StepResult:
    token: np.ndarray          # int32 [B, n]
    parent: np.ndarray         # int32 [B, n]
    depth: np.ndarray          # int32 [B, n]
    phat: np.ndarray           # float64 [B, n]
    n_sel: np.ndarray          # int32 [B]
    depth_reached: np.ndarray  # int32 [B]
    expected_len: np.ndarray   # float64 [B]
    esub_trace: np.ndarray     # float64 [B, max_depth]
    min_gap: np.ndarray        # float64 [B]
    stop_margin: np.ndarray    # float64 [B]
    mask: np.ndarray           # uint64 [B, n, W]
    position_ids: np.ndarray   # int32 [B, n]
    accept_len: np.ndarray     # int32 [B]
    accept_tokens: np.ndarray  # int32 [B, max_depth+1]
    accept_nodes: np.ndarray   # int32 [B, max_depth]
    next_root: np.ndarray      # int32 [B]


class Memo:
    """Row-result memo for parity runs on the table model (not for timing)."""

    def __init__(self, k: int, cap: int = 16384):
        self.handle = lib().ot_memo_create(cap, k)

    def __del__(self):
        if getattr(self, "handle", None):
            lib().ot_memo_destroy(self.handle)
            self.handle = None


def table_step(draft: np.ndarray, target: np.ndarray | None, root_token: np.ndarray, n: int, k: int,
               max_depth: int, delta: float, base_pos: np.ndarray | None = None,
               force_depth: np.ndarray | None = None, memo: Memo | None = None) -> StepResult:
    """One decoding step (build, mask, verify) for a batch on the table model."""
    H, V = draft.shape
    assert draft.dtype == np.uint16 and draft.flags.c_contiguous
    if target is not None:
        assert target.shape == draft.shape and target.dtype == np.uint16 and target.flags.c_contiguous
    root_token = np.ascontiguousarray(root_token, dtype=np.int32)
    B = root_token.shape[0]
    W = (n + 63) // 64
    if base_pos is not None:
        base_pos = np.ascontiguousarray(base_pos, dtype=np.int32)
    if force_depth is not None:
        force_depth = np.ascontiguousarray(force_depth, dtype=np.int32)
    r = StepResult(
        token=np.empty((B, n), np.int32), parent=np.empty((B, n), np.int32), depth=np.empty((B, n), np.int32),
        phat=np.empty((B, n), np.float64), n_sel=np.empty(B, np.int32), depth_reached=np.empty(B, np.int32),
        expected_len=np.empty(B, np.float64), esub_trace=np.zeros((B, max_depth), np.float64),
        min_gap=np.empty(B, np.float64), stop_margin=np.empty(B, np.float64),
        mask=np.zeros((B, n, W), np.uint64), position_ids=np.zeros((B, n), np.int32),
        accept_len=np.zeros(B, np.int32), accept_tokens=np.full((B, max_depth + 1), -1, np.int32),
        accept_nodes=np.full((B, max_depth), -1, np.int32), next_root=np.full(B, -1, np.int32))
    rc = lib().ot_table_step(
        _p(draft, C.c_uint16), _p(target, C.c_uint16), C.c_int32(H), C.c_int32(V),
        _p(root_token, C.c_int32), _p(base_pos, C.c_int32), C.c_int32(B),
        C.c_int32(n), C.c_int32(k), C.c_int32(max_depth), C.c_double(delta),
        _p(force_depth, C.c_int32), C.c_void_p(memo.handle if memo else None),
        _p(r.token, C.c_int32), _p(r.parent, C.c_int32), _p(r.depth, C.c_int32), _p(r.phat, C.c_double),
        _p(r.n_sel, C.c_int32), _p(r.depth_reached, C.c_int32), _p(r.expected_len, C.c_double),
        _p(r.esub_trace, C.c_double), _p(r.min_gap, C.c_double), _p(r.stop_margin, C.c_double),
        _p(r.mask, C.c_uint64), _p(r.position_ids, C.c_int32),
        _p(r.accept_len, C.c_int32), _p(r.accept_tokens, C.c_int32), _p(r.accept_nodes, C.c_int32),
        _p(r.next_root, C.c_int32))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return r


def table_build_rows(draft: np.ndarray, root_token: np.ndarray, n: int, k: int, max_depth: int, delta: float, prune: bool):
    """Trees of a batch on the table model, full or pruned (only layer nodes still among the n largest
    are drafted from), and the draft rows each sequence read.  Returns (StepResult-like dict, rows)."""
    H, V = draft.shape
    root_token = np.ascontiguousarray(root_token, dtype=np.int32)
    B = root_token.shape[0]
    out = dict(token=np.empty((B, n), np.int32), parent=np.empty((B, n), np.int32), depth=np.empty((B, n), np.int32),
               phat=np.empty((B, n), np.float64), n_sel=np.empty(B, np.int32), depth_reached=np.empty(B, np.int32),
               expected_len=np.empty(B, np.float64), esub_trace=np.zeros((B, max_depth), np.float64))
    rows = np.zeros(B, np.int64)
    rc = lib().ot_table_build_rows(
        _p(draft, C.c_uint16), C.c_int32(H), C.c_int32(V), _p(root_token, C.c_int32), C.c_int32(B),
        C.c_int32(n), C.c_int32(k), C.c_int32(max_depth), C.c_double(delta), C.c_int32(1 if prune else 0),
        _p(out["token"], C.c_int32), _p(out["parent"], C.c_int32), _p(out["depth"], C.c_int32), _p(out["phat"], C.c_double),
        _p(out["n_sel"], C.c_int32), _p(out["depth_reached"], C.c_int32), _p(out["expected_len"], C.c_double),
        _p(out["esub_trace"], C.c_double), _p(rows, C.c_int64))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return out, rows


def build_cb(logits_of, root_token: int, V: int, n: int, k: int, max_depth: int, delta: float,
             force_depth: int = 0):
    """Build one tree from a Python model: logits_of(root_token, path_tuple) -> sequence of V floats."""

    def _cb(_user, root, path, depth, out):
        vals = logits_of(int(root), tuple(int(path[i]) for i in range(depth)))
        for v in range(V):
            out[v] = float(vals[v])

    cb = LOGITS_FN(_cb)
    token = np.empty(n, np.int32); parent = np.empty(n, np.int32); depth = np.empty(n, np.int32)
    phat = np.empty(n, np.float64)
    n_sel = C.c_int32(); dr = C.c_int32(); ea = C.c_double(); mg = C.c_double(); sm = C.c_double()
    trace = np.zeros(max_depth, np.float64)
    rc = lib().ot_build_cb(cb, None, C.c_int32(root_token), C.c_int32(V), C.c_int32(n), C.c_int32(k),
                           C.c_int32(max_depth), C.c_double(delta), C.c_int32(force_depth),
                           _p(token, C.c_int32), _p(parent, C.c_int32), _p(depth, C.c_int32), _p(phat, C.c_double),
                           C.byref(n_sel), C.byref(dr), C.byref(ea), _p(trace, C.c_double), C.byref(mg), C.byref(sm))
    if rc != 0:
        raise ValueError("oracle: bad arguments")
    return dict(token=token, parent=parent, depth=depth, phat=phat, n_sel=n_sel.value, depth_reached=dr.value,
                expected_len=ea.value, esub_trace=trace, min_gap=mg.value, stop_margin=sm.value)


def verify_cb(logits_of, root_token: int, V: int, n_sel: int, max_depth: int, token, parent, depth):
    """Greedy acceptance walk with a Python target model (same callback form as build_cb)."""

    def _cb(_user, root, path, d, out):
        vals = logits_of(int(root), tuple(int(path[i]) for i in range(d)))
        for v in range(V):
            out[v] = float(vals[v])

    cb = LOGITS_FN(_cb)
    token = np.ascontiguousarray(token, np.int32); parent = np.ascontiguousarray(parent, np.int32)
    depth = np.ascontiguousarray(depth, np.int32)
    at = np.full(max_depth + 1, -1, np.int32); an = np.full(max_depth, -1, np.int32); nr = C.c_int32()
    A = lib().ot_verify_cb(cb, None, C.c_int32(root_token), C.c_int32(V), C.c_int32(n_sel), C.c_int32(max_depth),
                           _p(token, C.c_int32), _p(parent, C.c_int32), _p(depth, C.c_int32),
                           _p(at, C.c_int32), _p(an, C.c_int32), C.byref(nr))
    return dict(accept_len=int(A), accept_tokens=at, accept_nodes=an, next_root=nr.value)


def mask_of(parent, depth, n_sel: int, n: int, base_pos: int = 0):
    parent = np.ascontiguousarray(parent, np.int32); depth = np.ascontiguousarray(depth, np.int32)
    W = (n + 63) // 64
    mask = np.zeros((n, W), np.uint64); pos = np.zeros(n, np.int32)
    lib().ot_mask(_p(parent, C.c_int32), _p(depth, C.c_int32), C.c_int32(n_sel), C.c_int32(n), C.c_int32(base_pos),
                  _p(mask, C.c_uint64), _p(pos, C.c_int32))
    return mask, pos


def philox4x32_10(ctr, key):
    """The generator's block function: 4 x uint32 counter, 2 x uint32 key -> 4 x uint32."""
    c = np.ascontiguousarray(ctr, np.uint32); k = np.ascontiguousarray(key, np.uint32); o = np.zeros(4, np.uint32)
    lib().ot_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(o, C.c_uint32))
    return o


def uniform(seed: int, step: int, sequence: int, position: int) -> float:
    lib().ot_uniform.restype = C.c_double
    return float(lib().ot_uniform(C.c_uint64(seed), C.c_uint64(step), C.c_int32(sequence), C.c_int32(position)))


def sample_token(x: np.ndarray, tau: float, u: float):
    """(token, margin) of one inverse-CDF sample of softmax(x / tau)."""
    x = np.ascontiguousarray(x, np.float64)
    mg = C.c_double()
    lib().ot_sample_token.restype = C.c_int32
    y = lib().ot_sample_token(_p(x, C.c_double), C.c_int32(x.shape[0]), C.c_double(tau), C.c_double(u), C.byref(mg))
    return int(y), mg.value


def table_verify_sampled(target: np.ndarray, root_token, token, parent, depth, n_sel, max_depth: int, tau: float, seed: int, step: int):
    """Sampled verification of a batch of packed trees on the table model."""
    H, V = target.shape
    root_token = np.ascontiguousarray(root_token, np.int32)
    token = np.ascontiguousarray(token, np.int32); parent = np.ascontiguousarray(parent, np.int32)
    depth = np.ascontiguousarray(depth, np.int32); n_sel = np.ascontiguousarray(n_sel, np.int32)
    B, n = token.shape
    out = dict(accept_len=np.zeros(B, np.int32), accept_tokens=np.full((B, max_depth + 1), -1, np.int32),
               accept_nodes=np.full((B, max_depth), -1, np.int32), next_root=np.full(B, -1, np.int32),
               min_margin=np.zeros(B, np.float64))
    lib().ot_table_verify_sampled(
        _p(target, C.c_uint16), C.c_int32(H), C.c_int32(V), _p(root_token, C.c_int32), C.c_int32(B), C.c_int32(n),
        C.c_int32(max_depth), _p(token, C.c_int32), _p(parent, C.c_int32), _p(depth, C.c_int32), _p(n_sel, C.c_int32),
        C.c_double(tau), C.c_uint64(seed), C.c_uint64(step),
        _p(out["accept_len"], C.c_int32), _p(out["accept_tokens"], C.c_int32), _p(out["accept_nodes"], C.c_int32),
        _p(out["next_root"], C.c_int32), _p(out["min_margin"], C.c_double))
    return out


def dense_mask_of(parent, n_sel: int, n: int) -> np.ndarray:
    """[n+1][n+1] uint8: who attends to whom inside one step (position 0 = root, i+1 = node i)."""
    parent = np.ascontiguousarray(parent, np.int32)
    dense = np.zeros((n + 1, n + 1), np.uint8)
    lib().ot_dense_mask(_p(parent, C.c_int32), C.c_int32(n_sel), C.c_int32(n), _p(dense, C.c_uint8))
    return dense


def kv_keep_of(accept_nodes, accept_len: int, max_depth: int):
    """(gather [max_depth+1] int32, kept): the step positions whose keys and values stay cached, in path order."""
    an = np.ascontiguousarray(accept_nodes, np.int32)
    gather = np.empty(max_depth + 1, np.int32)
    lib().ot_kv_keep.restype = C.c_int32
    kept = lib().ot_kv_keep(_p(an, C.c_int32), C.c_int32(accept_len), C.c_int32(max_depth), _p(gather, C.c_int32))
    return gather, int(kept)


def row_softmax_topk(row_bf16: np.ndarray, k: int):
    """(tokens, probs, m, S) of one bf16 row."""
    row = np.ascontiguousarray(row_bf16, np.uint16)
    V = row.shape[0]
    kk = min(k, V)
    tok = np.empty(kk, np.int32); p = np.empty(kk, np.float64); m = C.c_double(); S = C.c_double()
    lib().ot_row_softmax_topk_bf16(_p(row, C.c_uint16), C.c_int32(V), C.c_int32(k),
                                   _p(tok, C.c_int32), _p(p, C.c_double), C.byref(m), C.byref(S))
    return tok, p, m.value, S.value


def row_argmax(row_bf16: np.ndarray) -> int:
    row = np.ascontiguousarray(row_bf16, np.uint16)
    return int(lib().ot_row_argmax_bf16(_p(row, C.c_uint16), C.c_int32(row.shape[0])))
