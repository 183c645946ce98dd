"""Thin ctypes binding of the C ABI in include/opt_tree.h.

Argument marshalling only: every step runs in the CUDA library.  PyTorch is used
for device memory and streams.  There is no CPU fallback: if the library is not
built or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libopt_tree.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_INTERNAL = 0, -1, -2, -3, -4, -5

EXPORTS = ["opt_tree_workspace_bytes", "opt_tree_create", "opt_tree_destroy", "opt_tree_build", "opt_tree_mask",
           "opt_tree_verify", "opt_tree_row_softmax_topk", "opt_tree_step_host", "opt_tree_last_device_status",
           "opt_tree_launch_count", "opt_tree_strerror", "opt_tree_verify_static", "opt_tree_post_verify", "opt_tree_build_pruned", "opt_tree_layers_begin",
           "opt_tree_layers_step", "opt_tree_verify_sampled", "opt_tree_selftest_waits"]


class Config(C.Structure):
    _fields_ = [(f, C.c_int32) for f in ("V", "H", "n", "k", "max_depth", "max_batch")]


class Out(C.Structure):
    _fields_ = [(f, C.c_void_p) for f in
                ("token", "parent", "depth", "phat", "n_sel", "depth_reached", "expected_len", "esub_trace")]


class HostOut(C.Structure):
    _fields_ = [(f, C.c_void_p) for f in
                ("token", "parent", "depth", "phat", "n_sel", "depth_reached", "expected_len", "mask", "position_ids",
                 "accept_len", "accept_tokens", "accept_nodes", "next_root")]


_lib = None


def lib():
    """Loads the shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2406_17276_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.opt_tree_workspace_bytes.restype = C.c_size_t
        L.opt_tree_workspace_bytes.argtypes = [C.POINTER(Config)]
        L.opt_tree_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Config)]
        L.opt_tree_destroy.argtypes = [C.c_void_p]
        L.opt_tree_build.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_float, C.POINTER(Out), C.c_void_p]
        L.opt_tree_mask.argtypes = [C.c_void_p, C.POINTER(Out), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.opt_tree_verify.argtypes = [C.c_void_p, C.POINTER(Out), C.c_void_p, C.c_void_p, C.c_int32,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.opt_tree_row_softmax_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                                C.c_void_p]
        L.opt_tree_step_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                         C.c_float, C.POINTER(HostOut), C.c_void_p]
        L.opt_tree_last_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
        L.opt_tree_launch_count.restype = C.c_int64
        L.opt_tree_launch_count.argtypes = [C.c_void_p]
        L.opt_tree_verify_static.argtypes = [C.POINTER(Config), C.POINTER(Out), C.c_void_p, C.c_void_p, C.c_int32,
                                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.opt_tree_build_pruned.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_float, C.POINTER(Out), C.c_void_p,
                                            C.c_void_p]
        L.opt_tree_verify_sampled.argtypes = [C.c_void_p, C.POINTER(Out), C.c_void_p, C.c_void_p, C.c_int32, C.c_double,
                                              C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.opt_tree_layers_begin.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.opt_tree_layers_step.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.POINTER(Out), C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_void_p]
        L.opt_tree_post_verify.argtypes = [C.c_void_p, C.POINTER(Out), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.opt_tree_selftest_waits.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.opt_tree_strerror.restype = C.c_char_p
        L.opt_tree_strerror.argtypes = [C.c_int]
        _lib = L
    return _lib


class OptTreeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib().opt_tree_strerror(code).decode()} ({code})")


def _check(code: int, where: str):
    if code != OK:
        raise OptTreeError(code, where)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(None)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class Tree:
    """Device tensors of one built batch (see opt_tree_out)."""
    token: torch.Tensor
    parent: torch.Tensor
    depth: torch.Tensor
    phat: torch.Tensor
    n_sel: torch.Tensor
    depth_reached: torch.Tensor
    expected_len: torch.Tensor
    esub_trace: torch.Tensor | None

    def c_struct(self) -> Out:
        return Out(*[t.data_ptr() if t is not None else None for t in
                     (self.token, self.parent, self.depth, self.phat, self.n_sel, self.depth_reached,
                      self.expected_len, self.esub_trace)])


class OptTree:
    """A library context: fixed (V, H, n, k, max_depth, max_batch), workspace allocated once."""

    def __init__(self, V: int, H: int, n: int, k: int, max_depth: int, max_batch: int, device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the OPT-Tree library has no CPU fallback")
        self.cfg = Config(V, H, n, k, max_depth, max_batch)
        self.device = torch.device(device)
        self.W = (n + 63) // 64
        self._ctx = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib().opt_tree_create(C.byref(self._ctx), C.byref(self.cfg)), "opt_tree_create")

    def close(self):
        if self._ctx:
            lib().opt_tree_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- allocation helpers (torch owns the memory) ----
    def alloc_tree(self, B: int, trace: bool = True) -> Tree:
        c, dev = self.cfg, self.device
        i32 = dict(dtype=torch.int32, device=dev)
        f64 = dict(dtype=torch.float64, device=dev)
        return Tree(torch.empty((B, c.n), **i32), torch.empty((B, c.n), **i32), torch.empty((B, c.n), **i32),
                    torch.empty((B, c.n), **f64), torch.empty(B, **i32), torch.empty(B, **i32), torch.empty(B, **f64),
                    torch.empty((B, c.max_depth), **f64) if trace else None)

    # ---- entry points (same names as the C ABI) ----
    def build(self, draft: torch.Tensor, root_token: torch.Tensor, delta: float, out: Tree | None = None) -> Tree:
        B = root_token.shape[0]
        out = out or self.alloc_tree(B)
        cs = out.c_struct()
        _check(lib().opt_tree_build(self._ctx, _ptr(draft), _ptr(root_token), B, C.c_float(delta), C.byref(cs), _stream()),
               "opt_tree_build")
        return out

    def build_pruned(self, draft: torch.Tensor, root_token: torch.Tensor, delta: float, out: Tree | None = None,
                     rows_read: torch.Tensor | None = None):
        """opt_tree_build_pruned: the same trees from fewer draft rows; returns (tree, rows_read [B] int32)."""
        B = root_token.shape[0]
        out = out or self.alloc_tree(B)
        if rows_read is None:
            rows_read = torch.empty(B, dtype=torch.int32, device=self.device)
        cs = out.c_struct()
        _check(lib().opt_tree_build_pruned(self._ctx, _ptr(draft), _ptr(root_token), B, C.c_float(delta), C.byref(cs),
                                           _ptr(rows_read), _stream()), "opt_tree_build_pruned")
        return out, rows_read

    def layers_begin(self, B: int):
        _check(lib().opt_tree_layers_begin(self._ctx, B, _stream()), "opt_tree_layers_begin")

    def layers_step(self, frontier_logits: torch.Tensor, delta: float, tree: Tree, nxt=None):
        """One layer of the layer-by-layer build; frontier_logits is [B][stride][V] bf16 bits on the device.
        Returns (next_tokens [B][n], next_parent [B][n], next_count [B])."""
        B, stride = frontier_logits.shape[0], frontier_logits.shape[1]
        if nxt is None:
            i32 = dict(dtype=torch.int32, device=self.device)
            nxt = (torch.empty((B, self.cfg.n), **i32), torch.empty((B, self.cfg.n), **i32), torch.empty(B, **i32))
        cs = tree.c_struct()
        _check(lib().opt_tree_layers_step(self._ctx, _ptr(frontier_logits), stride, B, C.c_float(delta), C.byref(cs),
                                          _ptr(nxt[0]), _ptr(nxt[1]), _ptr(nxt[2]), _stream()), "opt_tree_layers_step")
        return nxt

    def mask(self, tree: Tree, base_pos: torch.Tensor | None = None, mask: torch.Tensor | None = None,
             position_ids: torch.Tensor | None = None):
        B = tree.token.shape[0]
        if mask is None:
            mask = torch.empty((B, self.cfg.n, self.W), dtype=torch.int64, device=self.device)   # uint64 bit patterns
        if position_ids is None:
            position_ids = torch.empty((B, self.cfg.n), dtype=torch.int32, device=self.device)
        cs = tree.c_struct()
        _check(lib().opt_tree_mask(self._ctx, C.byref(cs), B, _ptr(base_pos), _ptr(mask), _ptr(position_ids), _stream()),
               "opt_tree_mask")
        return mask, position_ids

    def verify(self, tree: Tree, target: torch.Tensor, root_token: torch.Tensor, out=None):
        B = tree.token.shape[0]
        D = self.cfg.max_depth
        if out is None:
            i32 = dict(dtype=torch.int32, device=self.device)
            out = (torch.empty(B, **i32), torch.empty((B, D + 1), **i32), torch.empty((B, D), **i32), torch.empty(B, **i32))
        cs = tree.c_struct()
        _check(lib().opt_tree_verify(self._ctx, C.byref(cs), _ptr(target), _ptr(root_token), B,
                                     _ptr(out[0]), _ptr(out[1]), _ptr(out[2]), _ptr(out[3]), _stream()), "opt_tree_verify")
        return out

    def post_verify(self, tree: Tree, mask: torch.Tensor, accept_len: torch.Tensor, accept_nodes: torch.Tensor, out=None):
        """Dense (n+1)x(n+1) attention mask and the cache keep list of the accepted path."""
        B, n, D = tree.token.shape[0], self.cfg.n, self.cfg.max_depth
        if out is None:
            out = (torch.empty((B, n + 1, n + 1), dtype=torch.uint8, device=self.device),
                   torch.empty((B, D + 1), dtype=torch.int32, device=self.device),
                   torch.empty(B, dtype=torch.int32, device=self.device))
        cs = tree.c_struct()
        _check(lib().opt_tree_post_verify(self._ctx, C.byref(cs), _ptr(mask), _ptr(accept_len), _ptr(accept_nodes), B,
                                          _ptr(out[0]), _ptr(out[1]), _ptr(out[2]), _stream()), "opt_tree_post_verify")
        return out

    def verify_sampled(self, tree: Tree, target: torch.Tensor, root_token: torch.Tensor, tau: float, seed: int, step: int,
                       out=None):
        B = tree.token.shape[0]
        D = self.cfg.max_depth
        if out is None:
            i32 = dict(dtype=torch.int32, device=self.device)
            out = (torch.empty(B, **i32), torch.empty((B, D + 1), **i32), torch.empty((B, D), **i32), torch.empty(B, **i32))
        cs = tree.c_struct()
        _check(lib().opt_tree_verify_sampled(self._ctx, C.byref(cs), _ptr(target), _ptr(root_token), B, C.c_double(tau),
                                             C.c_uint64(seed), C.c_uint64(step), _ptr(out[0]), _ptr(out[1]), _ptr(out[2]),
                                             _ptr(out[3]), _stream()), "opt_tree_verify_sampled")
        return out

    def row_softmax_topk(self, logits: torch.Tensor, rows: torch.Tensor):
        nrows = rows.shape[0]
        tok = torch.empty((nrows, self.cfg.k), dtype=torch.int32, device=self.device)
        prob = torch.empty((nrows, self.cfg.k), dtype=torch.float64, device=self.device)
        _check(lib().opt_tree_row_softmax_topk(self._ctx, _ptr(logits), _ptr(rows), nrows, _ptr(tok), _ptr(prob), _stream()),
               "opt_tree_row_softmax_topk")
        return tok, prob

    def alloc_host_out(self, B: int) -> dict:
        """Pinned host buffers for step_host."""
        c = self.cfg
        def pin(shape, dt):
            return torch.empty(shape, dtype=dt).pin_memory()
        return dict(token=pin((B, c.n), torch.int32), parent=pin((B, c.n), torch.int32), depth=pin((B, c.n), torch.int32),
                    phat=pin((B, c.n), torch.float64), n_sel=pin((B,), torch.int32), depth_reached=pin((B,), torch.int32),
                    expected_len=pin((B,), torch.float64), mask=pin((B, c.n, self.W), torch.int64),
                    position_ids=pin((B, c.n), torch.int32), accept_len=pin((B,), torch.int32),
                    accept_tokens=pin((B, c.max_depth + 1), torch.int32), accept_nodes=pin((B, c.max_depth), torch.int32),
                    next_root=pin((B,), torch.int32))

    def step_host(self, draft: torch.Tensor, target: torch.Tensor, root_token_host: torch.Tensor,
                  base_pos_host: torch.Tensor | None, delta: float, host_out: dict) -> dict:
        B = root_token_host.shape[0]
        ho = HostOut(*[host_out[f].data_ptr() for f, _ in HostOut._fields_])
        _check(lib().opt_tree_step_host(self._ctx, _ptr(draft), _ptr(target), _ptr(root_token_host), _ptr(base_pos_host),
                                        B, C.c_float(delta), C.byref(ho), _stream()), "opt_tree_step_host")
        return host_out

    def selftest_waits(self) -> torch.Tensor:
        """opt_tree_selftest_waits: one status word per kind of bounded wait (each should read ERR_TIMEOUT)."""
        res = torch.full((5,), 77, dtype=torch.int32, device=self.device)
        _check(lib().opt_tree_selftest_waits(self._ctx, _ptr(res), _stream()), "opt_tree_selftest_waits")
        return res

    def device_status(self) -> int:
        st = C.c_int32(0)
        _check(lib().opt_tree_last_device_status(self._ctx, C.byref(st)), "opt_tree_last_device_status")
        return st.value

    def launch_count(self) -> int:
        return int(lib().opt_tree_launch_count(self._ctx))


def verify_static(cfg: Config, tree: Tree, target: torch.Tensor, root_token: torch.Tensor, out, device_status: torch.Tensor | None = None):
    """opt_tree_verify_static: verification for callers that cannot allocate.  Needs no OptTree context; every
    buffer, outputs included, is the caller's (out = (accept_len, accept_tokens, accept_nodes, next_root))."""
    B = tree.token.shape[0]
    cs = tree.c_struct()
    _check(lib().opt_tree_verify_static(C.byref(cfg), C.byref(cs), _ptr(target), _ptr(root_token), B, _ptr(out[0]), _ptr(out[1]),
                                        _ptr(out[2]), _ptr(out[3]), _ptr(device_status), _stream()), "opt_tree_verify_static")
    return out
