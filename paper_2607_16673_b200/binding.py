"""Thin Python binding of libspeca's C ABI (``include/speca.h``).

Argument marshalling only: every function takes CUDA ``torch`` tensors (bf16 tensors
for q, k, v; int32 for topology), checks shapes and dtypes, and passes raw device
pointers plus the current CUDA stream to the entry point of the same name.  Nothing
is computed here and there is no fallback: if ``libspeca.so`` has not been built
(``python -m paper_2607_16673_b200.build``) every call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspeca.so")

OK = 0
STATUS_BAD_PARENT, STATUS_BAD_OFFSETS, STATUS_BAD_PATH, STATUS_TOO_DEEP = 1, 2, 4, 8
STATUS_TOO_MANY, STATUS_TIMEOUT, STATUS_BAD_DEPTH = 16, 32, 64
ROUTE_AUTO, ROUTE_SERIAL, ROUTE_FACTORIZED, ROUTE_TF32, ROUTE_EFFECTIVE = 0, 1, 2, 3, 4
RULE_GATED_DELTA, RULE_GATED_NO_ERASE = 0, 1

EXPORTS = ["speca_version", "speca_strerror", "speca_workspace_bytes", "speca_decode_step",
           "speca_verify_chain", "speca_verify_tree", "speca_greedy_accept", "speca_commit",
           "speca_verify_tree_noalloc", "speca_commit_verify_tree", "speca_commit_conv",
           "speca_tree_mask_to_parent", "speca_prune_tree", "speca_stochastic_accept",
           "speca_chain_decompose"]
NOALLOC_MAX_BATCH, NOALLOC_MAX_NODES = 256, 16384


class SpecaError(RuntimeError):
    pass


class _Dims(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("heads", ctypes.c_int32),
                ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32), ("scale", ctypes.c_float),
                ("max_depth", ctypes.c_int32), ("max_nodes", ctypes.c_int32), ("route", ctypes.c_int32),
                ("rule", ctypes.c_int32)]


@dataclass
class Dims:
    n_layers: int
    batch: int
    heads: int
    d_k: int
    d_v: int
    scale: float = 1.0
    max_depth: int = 8
    max_nodes: int = 64
    route: int = ROUTE_AUTO
    rule: int = 0

    def c(self) -> _Dims:
        return _Dims(self.n_layers, self.batch, self.heads, self.d_k, self.d_v, self.scale,
                     self.max_depth, self.max_nodes, self.route, self.rule)


_lib = None


def lib() -> ctypes.CDLL:
    """Load libspeca.so; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise SpecaError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_16673_b200.build` "
                             "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        dp = ctypes.POINTER(_Dims)
        L.speca_version.restype = ctypes.c_int
        L.speca_strerror.restype = ctypes.c_char_p
        L.speca_strerror.argtypes = [ctypes.c_int]
        L.speca_workspace_bytes.restype = sz
        L.speca_workspace_bytes.argtypes = [dp, i32]
        L.speca_decode_step.argtypes = [dp] + [vp] * 8
        L.speca_verify_chain.argtypes = [dp] + [vp] * 7 + [i32, vp, vp, vp, sz, vp, vp]
        L.speca_verify_tree.argtypes = [dp] + [vp] * 7 + [i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.speca_verify_tree_noalloc.argtypes = [dp] + [vp] * 7 + [i32, vp, vp, vp, vp, vp, vp]
        L.speca_greedy_accept.argtypes = [i32, i32] + [vp] * 10
        L.speca_commit.argtypes = [dp] + [vp] * 6 + [i32] + [vp] * 5
        L.speca_commit_verify_tree.argtypes = ([dp] + [vp] * 7 + [i32] + [vp] * 3 + [vp] * 6 + [i32] + [vp] * 5 +
                                               [sz, vp, vp])
        L.speca_commit_conv.argtypes = [i32] * 5 + [vp, vp, vp, i32, vp, vp, vp, vp]
        L.speca_tree_mask_to_parent.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        L.speca_tree_mask_to_parent.restype = ctypes.c_int
        L.speca_prune_tree.argtypes = [i32, i32, ctypes.c_float, i32] + [vp] * 8
        L.speca_prune_tree.restype = ctypes.c_int
        L.speca_stochastic_accept.argtypes = [i32, i32] + [vp] * 9
        L.speca_chain_decompose.argtypes = [i32, i32] + [vp] * 6
        L.speca_chain_decompose.restype = ctypes.c_int
        L.speca_stochastic_accept.restype = ctypes.c_int
        for name in ("speca_decode_step", "speca_verify_chain", "speca_verify_tree", "speca_greedy_accept",
                     "speca_commit", "speca_verify_tree_noalloc", "speca_commit_verify_tree", "speca_commit_conv"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise SpecaError(f"{what}: {lib().speca_strerror(rc).decode()} (code {rc})")


def _ptr(t: Optional[torch.Tensor], dtype, shape=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise SpecaError(f"{name}: need a contiguous CUDA tensor of dtype {dtype}, got {t.dtype} on {t.device}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise SpecaError(f"{name}: shape {tuple(t.shape)} != expected {tuple(shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def version() -> int:
    return int(lib().speca_version())


def workspace_bytes(dims: Dims, total_nodes: int) -> int:
    d = dims.c()
    return int(lib().speca_workspace_bytes(ctypes.byref(d), int(total_nodes)))


def alloc_workspace(dims: Dims, total_nodes: int, device="cuda") -> torch.Tensor:
    return torch.empty(workspace_bytes(dims, total_nodes), dtype=torch.uint8, device=device)


def decode_step(dims: Dims, S, q, k, v, alpha, beta, o) -> None:
    L, B, H, dk, dv = dims.n_layers, dims.batch, dims.heads, dims.d_k, dims.d_v
    d = dims.c()
    rc = lib().speca_decode_step(
        ctypes.byref(d), _ptr(S, torch.float32, (L, B, H, dv, dk), "S"),
        _ptr(q, torch.bfloat16, (L, B, H, dk), "q"), _ptr(k, torch.bfloat16, (L, B, H, dk), "k"),
        _ptr(v, torch.bfloat16, (L, B, H, dv), "v"), _ptr(alpha, torch.float32, (L, B, H), "alpha"),
        _ptr(beta, torch.float32, (L, B, H), "beta"), _ptr(o, torch.float32, (L, B, H, dv), "o"), _stream())
    _check(rc, "speca_decode_step")


def _verify_args(dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, o, u):
    L, B, H, dk, dv, T = dims.n_layers, dims.batch, dims.heads, dims.d_k, dims.d_v, int(total_nodes)
    return [_ptr(S0, torch.float32, (L, B, H, dv, dk), "S0"), _ptr(q, torch.bfloat16, (L, T, H, dk), "q"),
            _ptr(k, torch.bfloat16, (L, T, H, dk), "k"), _ptr(v, torch.bfloat16, (L, T, H, dv), "v"),
            _ptr(alpha, torch.float32, (L, T, H), "alpha"), _ptr(beta, torch.float32, (L, T, H), "beta"),
            _ptr(node_offsets, torch.int32, (B + 1,), "node_offsets")], \
           [_ptr(o, torch.float32, (L, T, H, dv), "o"), _ptr(u, torch.float32, (L, T, H, dv), "u")]


def verify_chain(dims: Dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, o, u, workspace, status) -> None:
    ins, outs = _verify_args(dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, o, u)
    d = dims.c()
    rc = lib().speca_verify_chain(ctypes.byref(d), *ins, int(total_nodes), *outs,
                                  _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(),
                                  _ptr(status, torch.int32, (1,), "status"), _stream())
    _check(rc, "speca_verify_chain")


def verify_tree(dims: Dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, parent, depth, o, u,
                workspace, status) -> None:
    ins, outs = _verify_args(dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, o, u)
    T = int(total_nodes)
    d = dims.c()
    rc = lib().speca_verify_tree(ctypes.byref(d), *ins, T, _ptr(parent, torch.int32, (T,), "parent"),
                                 _ptr(depth, torch.int32, (T,), "depth"), *outs,
                                 _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(),
                                 _ptr(status, torch.int32, (1,), "status"), _stream())
    _check(rc, "speca_verify_tree")


def verify_tree_noalloc(dims: Dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, parent, depth, o, u,
                        status) -> None:
    """speca_verify_tree without a workspace argument, for callers that may not allocate device
    memory: the scratch is a fixed array inside the library (batch <= NOALLOC_MAX_BATCH,
    total_nodes <= NOALLOC_MAX_NODES).  Calls on one device share that array, so calls that
    could overlap on the GPU must be ordered by the caller."""
    ins, outs = _verify_args(dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, o, u)
    T = int(total_nodes)
    d = dims.c()
    rc = lib().speca_verify_tree_noalloc(ctypes.byref(d), *ins, T, _ptr(parent, torch.int32, (T,), "parent"),
                                         _ptr(depth, torch.int32, (T,), "depth"), *outs,
                                         _ptr(status, torch.int32, (1,), "status"), _stream())
    _check(rc, "speca_verify_tree_noalloc")


def greedy_accept(batch: int, max_depth: int, node_offsets, parent, draft_tok, target_tok, root_target_tok,
                  path_idx, path_len, next_tok, status) -> None:
    i32 = torch.int32
    rc = lib().speca_greedy_accept(
        int(batch), int(max_depth), _ptr(node_offsets, i32, (batch + 1,), "node_offsets"),
        _ptr(parent, i32, None, "parent"), _ptr(draft_tok, i32, tuple(parent.shape), "draft_tok"),
        _ptr(target_tok, i32, tuple(parent.shape), "target_tok"),
        _ptr(root_target_tok, i32, (batch,), "root_target_tok"),
        _ptr(path_idx, i32, (batch, max_depth), "path_idx"), _ptr(path_len, i32, (batch,), "path_len"),
        _ptr(next_tok, i32, (batch,), "next_tok"), _ptr(status, i32, (1,), "status"), _stream())
    _check(rc, "speca_greedy_accept")


def stochastic_accept(batch: int, max_depth: int, node_offsets, parent, p_target, p_draft, uniform,
                      path_idx, path_len, status) -> None:
    """speca_stochastic_accept: the walk over first passing children (uniform * p_draft < p_target)."""
    i32, f32 = torch.int32, torch.float32
    shape = tuple(parent.shape)
    rc = lib().speca_stochastic_accept(
        int(batch), int(max_depth), _ptr(node_offsets, i32, (batch + 1,), "node_offsets"),
        _ptr(parent, i32, None, "parent"), _ptr(p_target, f32, shape, "p_target"),
        _ptr(p_draft, f32, shape, "p_draft"), _ptr(uniform, f32, shape, "uniform"),
        _ptr(path_idx, i32, (batch, max_depth), "path_idx"), _ptr(path_len, i32, (batch,), "path_len"),
        _ptr(status, i32, (1,), "status"), _stream())
    _check(rc, "speca_stochastic_accept")


def commit(dims: Dims, S, k, v, alpha, beta, node_offsets, total_nodes, parent, path_idx, path_len, status) -> None:
    L, B, H, dk, dv, T = dims.n_layers, dims.batch, dims.heads, dims.d_k, dims.d_v, int(total_nodes)
    i32 = torch.int32
    d = dims.c()
    rc = lib().speca_commit(
        ctypes.byref(d), _ptr(S, torch.float32, (L, B, H, dv, dk), "S"),
        _ptr(k, torch.bfloat16, (L, T, H, dk), "k"), _ptr(v, torch.bfloat16, (L, T, H, dv), "v"),
        _ptr(alpha, torch.float32, (L, T, H), "alpha"), _ptr(beta, torch.float32, (L, T, H), "beta"),
        _ptr(node_offsets, i32, (B + 1,), "node_offsets"), T, _ptr(parent, i32, (T,), "parent"),
        _ptr(path_idx, i32, (B, dims.max_depth), "path_idx"), _ptr(path_len, i32, (B,), "path_len"),
        _ptr(status, i32, (1,), "status"), _stream())
    _check(rc, "speca_commit")


def commit_verify_tree(dims: Dims, S, prev, path_idx, path_len, q, k, v, alpha, beta, node_offsets, total_nodes,
                       parent, depth, o, u, workspace, status) -> None:
    """speca_commit_verify_tree: commit the previous draft's accepted paths into S and verify the
    new draft from the committed state.  ``prev`` is None (nothing pending) or a dict with the
    previous draft's ``k, v, alpha, beta`` records, ``u`` (what its verification wrote, or None),
    ``node_offsets``, ``total_nodes`` and ``parent`` (or None)."""
    L, B, H, dk, dv, T = dims.n_layers, dims.batch, dims.heads, dims.d_k, dims.d_v, int(total_nodes)
    i32 = torch.int32
    if prev is None:
        pargs = [None] * 5 + [None, 0, None]
        Tp = 0
    else:
        Tp = int(prev["total_nodes"])
        pargs = [_ptr(prev["k"], torch.bfloat16, (L, Tp, H, dk), "k_prev"),
                 _ptr(prev["v"], torch.bfloat16, (L, Tp, H, dv), "v_prev"),
                 _ptr(prev["alpha"], torch.float32, (L, Tp, H), "alpha_prev"),
                 _ptr(prev["beta"], torch.float32, (L, Tp, H), "beta_prev"),
                 _ptr(prev.get("u"), torch.float32, (L, Tp, H, dv), "u_prev"),
                 _ptr(prev["node_offsets"], i32, (B + 1,), "node_offsets_prev"), Tp,
                 _ptr(prev.get("parent"), i32, (Tp,), "parent_prev")]
    d = dims.c()
    rc = lib().speca_commit_verify_tree(
        ctypes.byref(d), _ptr(S, torch.float32, (L, B, H, dv, dk), "S"), *pargs,
        _ptr(path_idx, i32, (B, dims.max_depth), "path_idx"), _ptr(path_len, i32, (B,), "path_len"),
        _ptr(q, torch.bfloat16, (L, T, H, dk), "q"), _ptr(k, torch.bfloat16, (L, T, H, dk), "k"),
        _ptr(v, torch.bfloat16, (L, T, H, dv), "v"), _ptr(alpha, torch.float32, (L, T, H), "alpha"),
        _ptr(beta, torch.float32, (L, T, H), "beta"), _ptr(node_offsets, i32, (B + 1,), "node_offsets"), T,
        _ptr(parent, i32, (T,), "parent"), _ptr(depth, i32, (T,), "depth"),
        _ptr(o, torch.float32, (L, T, H, dv), "o"), _ptr(u, torch.float32, (L, T, H, dv), "u"),
        _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(),
        _ptr(status, i32, (1,), "status"), _stream())
    _check(rc, "speca_commit_verify_tree")


def commit_conv(C, x, node_offsets, total_nodes, path_idx, path_len, status) -> None:
    """speca_commit_conv: shift the inputs of the accepted nodes into the convolution state.
    C bf16 [L,B,W,channels] (in place), x bf16 [L,T,channels]."""
    L, B, W, ch = C.shape
    T = int(total_nodes)
    i32 = torch.int32
    rc = lib().speca_commit_conv(
        int(L), int(B), int(ch), int(W), int(path_idx.shape[1]), _ptr(C, torch.bfloat16, (L, B, W, ch), "C"),
        _ptr(x, torch.bfloat16, (L, T, ch), "x"), _ptr(node_offsets, i32, (B + 1,), "node_offsets"), T,
        _ptr(path_idx, i32, (B, path_idx.shape[1]), "path_idx"), _ptr(path_len, i32, (B,), "path_len"),
        _ptr(status, i32, (1,), "status"), _stream())
    _check(rc, "speca_commit_conv")


def tree_mask_to_parent(mask, node_offsets, parent, status) -> None:
    """speca_tree_mask_to_parent: mask uint8 [B,N,N] -> parent int32 [T] (written in place)."""
    B, N, N2 = mask.shape
    assert N == N2
    rc = lib().speca_tree_mask_to_parent(int(B), int(N), _ptr(mask, torch.uint8, (B, N, N), "mask"),
                                         _ptr(node_offsets, torch.int32, (B + 1,), "node_offsets"),
                                         _ptr(parent, torch.int32, None, "parent"),
                                         _ptr(status, torch.int32, (1,), "status"), _stream())
    _check(rc, "speca_tree_mask_to_parent")


def prune_tree(max_nodes: int, tau: float, budget: int, node_offsets, parent, logp, out_offsets, out_parent,
               out_index, status) -> None:
    """speca_prune_tree: keep the nodes within tau of the best cumulative log-probability, at most
    `budget` per sequence; packed outputs."""
    i32 = torch.int32
    B = node_offsets.numel() - 1
    T = parent.numel()
    rc = lib().speca_prune_tree(int(B), int(max_nodes), float(tau), int(budget),
                                _ptr(node_offsets, i32, (B + 1,), "node_offsets"), _ptr(parent, i32, (T,), "parent"),
                                _ptr(logp, torch.float32, (T,), "logp"), _ptr(out_offsets, i32, (B + 1,), "out_offsets"),
                                _ptr(out_parent, i32, (T,), "out_parent"), _ptr(out_index, i32, (T,), "out_index"),
                                _ptr(status, i32, (1,), "status"), _stream())
    _check(rc, "speca_prune_tree")


def chain_decompose(max_nodes: int, node_offsets, parent, chain_head, n_chains, status) -> None:
    """speca_chain_decompose: heavy-light chains; chain_head[t] = first node of t's chain, n_chains per sequence."""
    i32 = torch.int32
    B = node_offsets.numel() - 1
    T = parent.numel()
    rc = lib().speca_chain_decompose(int(B), int(max_nodes), _ptr(node_offsets, i32, (B + 1,), "node_offsets"),
                                     _ptr(parent, i32, (T,), "parent"), _ptr(chain_head, i32, (T,), "chain_head"),
                                     _ptr(n_chains, i32, (B,), "n_chains"), _ptr(status, i32, (1,), "status"), _stream())
    _check(rc, "speca_chain_decompose")
