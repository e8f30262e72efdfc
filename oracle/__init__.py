"""fp64 CPU oracle for the GDN speculative verify / accept / commit path.

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package.  It shares no code with
the CUDA library and never imports it.

The arithmetic lives in ``gdn_oracle.c`` (plain C, fp64, the definitions of
Sections 2.2, 4.2 and 5.1 written out).  This module compiles that file with
gcc on first use and exposes numpy-in / numpy-out wrappers.

Five small definitions are written here in numpy because they move or compare
values and compute nothing in floating point beyond fp32 additions in a fixed
order: ``commit_conv`` (convolution state, Section 7), ``tree_mask_to_parent``
(proposal converter, Section 7), ``prune_tree`` (confidence-guided pruning,
Section 6.1), ``stochastic_accept`` (the rejection-sampling-style rule of
Section 2.1 as a walk over per-node tests) and ``chain_decompose`` (the
heavy-light chains of Section 4.3).  Pins (tests/test_oracle_pins.py): hand cases and the causal-
convolution identity for the first, a round trip through independently built
masks for the second, a hand-worked example plus an independent sort-based
selection in fp64 on exactly representable scores for the third, hand cases, the
chain's closed-form acceptance-length distribution and an independent
level-by-level formulation for the fourth, the chains the paper prints for its
example (Section 4.3), the partition and path properties and the logarithmic
bound on chain changes along a root path for the fifth.  The rule
switch (``set_rule``) is pinned by the closed form of gated linear attention.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gdn_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libgdn_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, -O2, OpenMP).  Returns the path of the shared object."""
    with _lock:
        stale = (not os.path.exists(_LIB_PATH)
                 or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC))
        if force or stale:
            tmp = _LIB_PATH + f".tmp{os.getpid()}"
            # -ffp-contract=off: no fused multiply-add, every product is rounded
            # to fp64 before it is added, as written in the source.
            cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC",
                   "-shared", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB_PATH)
        i32, f64, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_rule.argtypes = [i32]
        lib.oracle_set_rule.restype = None
        lib.oracle_decode_step.argtypes = [i32] * 5 + [f64] + [vp] * 7
        lib.oracle_verify_tree.argtypes = [i32] * 5 + [f64] + [vp] * 9
        lib.oracle_greedy_accept.argtypes = [i32, i32] + [vp] * 8
        lib.oracle_commit.argtypes = [i32] * 6 + [vp] * 8
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


RULE_GATED_DELTA, RULE_GATED_NO_ERASE = 0, 1


def set_rule(rule: int) -> None:
    """Select the recurrence for the following calls: RULE_GATED_DELTA (default; DeltaNet is its alpha = 1
    case) or RULE_GATED_NO_ERASE, S' = alpha S + beta v k^T (GLA-style layers; Section 5.1, remark)."""
    _load().oracle_set_rule(int(rule))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    """Threads the loops over independent units may use (for timing; results do not depend on it)."""
    _load().oracle_set_num_threads(int(n))


def decode_step(S, q, k, v, alpha, beta, scale: float = 1.0):
    """One token per sequence.  S [L,B,H,dv,dk]; q,k uint16 [L,B,H,dk]; v uint16 [L,B,H,dv].

    Returns (S_new float64, o float64 [L,B,H,dv]).  The input is not modified.
    """
    S = np.array(S, dtype=np.float64, order="C", copy=True)
    L, B, H, dv, dk = S.shape
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    alpha, beta = _c(alpha, np.float32), _c(beta, np.float32)
    assert q.shape == (L, B, H, dk) and k.shape == (L, B, H, dk) and v.shape == (L, B, H, dv)
    assert alpha.shape == (L, B, H) and beta.shape == (L, B, H)
    o = np.empty((L, B, H, dv), dtype=np.float64)
    rc = _load().oracle_decode_step(L, B, H, dk, dv, float(scale), _p(S), _p(q), _p(k), _p(v),
                                    _p(alpha), _p(beta), _p(o))
    assert rc == 0
    return S, o


def verify_tree(S0, q, k, v, alpha, beta, node_offsets, parent, scale: float = 1.0):
    """Outputs of every draft node.  Returns o float64 [L,T,H,dv]."""
    S0 = _c(S0, np.float64)
    L, B, H, dv, dk = S0.shape
    node_offsets, parent = _c(node_offsets, np.int32), _c(parent, np.int32)
    T = int(node_offsets[B])
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    alpha, beta = _c(alpha, np.float32), _c(beta, np.float32)
    assert node_offsets.shape == (B + 1,) and parent.shape == (T,)
    assert q.shape == (L, T, H, dk) and k.shape == (L, T, H, dk) and v.shape == (L, T, H, dv)
    assert alpha.shape == (L, T, H) and beta.shape == (L, T, H)
    o = np.zeros((L, T, H, dv), dtype=np.float64)
    rc = _load().oracle_verify_tree(L, B, H, dk, dv, float(scale), _p(S0), _p(q), _p(k), _p(v),
                                    _p(alpha), _p(beta), _p(node_offsets), _p(parent), _p(o))
    if rc != 0:
        raise ValueError(f"oracle_verify_tree: bad topology (code {rc})")
    return o


def verify_chain(S0, q, k, v, alpha, beta, node_offsets, scale: float = 1.0):
    """Chain special case: parent[i] = i - 1 inside every sequence."""
    node_offsets = _c(node_offsets, np.int32)
    parent = np.concatenate([np.arange(-1, int(n) - 1, dtype=np.int32)
                             for n in np.diff(node_offsets)] + [np.zeros(0, np.int32)])
    return verify_tree(S0, q, k, v, alpha, beta, node_offsets, parent, scale)


def greedy_accept(node_offsets, parent, draft_tok, target_tok, root_target_tok, max_depth: int):
    """Returns (path_idx int32 [B,max_depth], path_len int32 [B], next_tok int32 [B])."""
    node_offsets, parent = _c(node_offsets, np.int32), _c(parent, np.int32)
    draft_tok, target_tok = _c(draft_tok, np.int32), _c(target_tok, np.int32)
    root_target_tok = _c(root_target_tok, np.int32)
    B = node_offsets.shape[0] - 1
    path_idx = np.empty((B, max_depth), dtype=np.int32)
    path_len = np.empty((B,), dtype=np.int32)
    next_tok = np.empty((B,), dtype=np.int32)
    rc = _load().oracle_greedy_accept(B, int(max_depth), _p(node_offsets), _p(parent),
                                      _p(draft_tok), _p(target_tok), _p(root_target_tok),
                                      _p(path_idx), _p(path_len), _p(next_tok))
    if rc != 0:
        raise ValueError(f"oracle_greedy_accept: code {rc}")
    return path_idx, path_len, next_tok


def commit(S, k, v, alpha, beta, node_offsets, path_idx, path_len):
    """Advance the state over the accepted records.  Returns S_new float64 (input untouched)."""
    S = np.array(S, dtype=np.float64, order="C", copy=True)
    L, B, H, dv, dk = S.shape
    node_offsets = _c(node_offsets, np.int32)
    path_idx, path_len = _c(path_idx, np.int32), _c(path_len, np.int32)
    T = int(node_offsets[B])
    max_depth = path_idx.shape[1]
    k, v = _c(k, np.uint16), _c(v, np.uint16)
    alpha, beta = _c(alpha, np.float32), _c(beta, np.float32)
    assert k.shape == (L, T, H, dk) and v.shape == (L, T, H, dv)
    assert alpha.shape == (L, T, H) and beta.shape == (L, T, H)
    assert path_idx.shape == (B, max_depth) and path_len.shape == (B,)
    rc = _load().oracle_commit(L, B, H, dk, dv, max_depth, _p(S), _p(k), _p(v), _p(alpha), _p(beta),
                               _p(node_offsets), _p(path_idx), _p(path_len))
    if rc != 0:
        raise ValueError(f"oracle_commit: bad path (code {rc})")
    return S


def commit_conv(C, x, node_offsets, path_idx, path_len):
    """Convolution state of the causal depthwise convolution in front of the GDN layer (Section 7: the
    state holder keeps (S, C)).  C [L,B,W,channels] are the last W = kernel_size - 1 inputs of every
    channel, oldest first; x [L,T,channels] the inputs of the draft nodes.  Feeding the accepted nodes
    through the convolution one by one shifts the register by one and appends the node's input; that
    is done here literally, token by token.  16-bit patterns are moved, never interpreted.
    Returns the new C (the input is not modified)."""
    C = np.array(C, copy=True)
    L, B, W, ch = C.shape
    node_offsets = _c(node_offsets, np.int32)
    path_idx, path_len = _c(path_idx, np.int32), _c(path_len, np.int32)
    assert x.shape[0] == L and x.shape[2] == ch and x.dtype == C.dtype
    for b in range(B):
        base, n = int(node_offsets[b]), int(node_offsets[b + 1] - node_offsets[b])
        for d in range(int(path_len[b])):
            t = int(path_idx[b, d])
            if not 0 <= t < n:
                raise ValueError("commit_conv: bad path")
            for l in range(L):
                for w in range(W - 1):
                    C[l, b, w] = C[l, b, w + 1]
                C[l, b, W - 1] = x[l, base + t]
    return C


def tree_mask_to_parent(mask, node_offsets):
    """Proposal converter (Section 7): a drafter's tree attention mask -> parent array.  mask uint8
    [B,N,N]; for sequence b with n nodes, mask[b,i,j] != 0 (i, j < n) iff node j is node i itself or one
    of its ancestors.  The parent of i is its deepest strict ancestor, i.e. the one with the most
    ancestors of its own; no strict ancestor -> -1.  Returns parent int32 [T] (local indices)."""
    node_offsets = _c(node_offsets, np.int32)
    B = node_offsets.shape[0] - 1
    out = np.full(int(node_offsets[B]), -1, np.int32)
    for b in range(B):
        base, n = int(node_offsets[b]), int(node_offsets[b + 1] - node_offsets[b])
        m = np.asarray(mask[b, :n, :n]) != 0
        size = m.sum(axis=1)
        for i in range(n):
            best = -1
            for j in range(n):
                if j != i and m[i, j] and (best < 0 or size[j] > size[best]):
                    best = j
            out[base + i] = best
    return out


def prune_tree(node_offsets, parent, logp, tau, budget):
    """Confidence-guided tree pruning (Section 6.1).  q(v) = sum of the step log-probabilities on the
    root path of v (fp32, added root first); q* = max q; the window keeps q(v) >= q* - tau; of the
    window the `budget` best by q are kept (ties: lower index first); a node whose parent was dropped is
    dropped too, so the result is ancestor-closed whatever the scores.  Returns (out_offsets int32 [B+1],
    out_parent int32 [T'], out_index int32 [T']): the kept nodes of every sequence in their original
    order, parents re-indexed, and each kept node's original local index."""
    node_offsets, parent = _c(node_offsets, np.int32), _c(parent, np.int32)
    logp = _c(logp, np.float32)
    B = node_offsets.shape[0] - 1
    offs, out_parent, out_index = [0], [], []
    for b in range(B):
        base, n = int(node_offsets[b]), int(node_offsets[b + 1] - node_offsets[b])
        par = parent[base:base + n]
        q = np.zeros(n, np.float32)
        for i in range(n):
            q[i] = np.float32((q[par[i]] if par[i] >= 0 else np.float32(0)) + logp[base + i])
        keep = np.zeros(n, bool)
        if n:
            thr = np.float32(q.max() - np.float32(tau))
            window = [i for i in range(n) if q[i] >= thr]
            window.sort(key=lambda i: (-float(q[i]), i))
            keep[window[:max(int(budget), 0)]] = True
            for i in range(n):
                if par[i] >= 0 and not keep[par[i]]:
                    keep[i] = False
        new = np.cumsum(keep) - 1
        for i in range(n):
            if keep[i]:
                out_parent.append(-1 if par[i] < 0 else int(new[par[i]]))
                out_index.append(i)
        offs.append(len(out_parent))
    return np.asarray(offs, np.int32), np.asarray(out_parent, np.int32), np.asarray(out_index, np.int32)


def stochastic_accept(node_offsets, parent, p_target, p_draft, uniform, max_depth: int):
    """Stochastic posterior selection (the rejection-sampling-style rule of Section 2.1) given per-node
    probabilities, as the plain walk: from the committed state, look at the children of the current
    node in ascending index; child t passes iff uniform[t] * p_draft[t] < p_target[t] (fp32 product,
    i.e. uniform < min(1, p_target / p_draft)); move to the first child that passes; stop when none
    does (a path longer than max_depth is outside the contract and raises).  Returns (path_idx int32 [B, max_depth] padded with -1,
    path_len int32 [B])."""
    node_offsets, parent = _c(node_offsets, np.int32), _c(parent, np.int32)
    p_target, p_draft, uniform = _c(p_target, np.float32), _c(p_draft, np.float32), _c(uniform, np.float32)
    B = node_offsets.shape[0] - 1
    path_idx = np.full((B, int(max_depth)), -1, np.int32)
    path_len = np.zeros(B, np.int32)
    for b in range(B):
        base, n = int(node_offsets[b]), int(node_offsets[b + 1] - node_offsets[b])
        cur, d = -1, 0
        while True:
            nxt = -1
            for t in range(cur + 1, n):
                if parent[base + t] == cur and np.float32(uniform[base + t] * p_draft[base + t]) < p_target[base + t]:
                    nxt = t
                    break
            if nxt < 0:
                break
            if d == max_depth:
                raise ValueError("accepted path longer than max_depth")
            path_idx[b, d] = nxt
            cur, d = nxt, d + 1
        path_len[b] = d
    return path_idx, path_len


def chain_decompose(node_offsets, parent):
    """Heavy-light chain decomposition (Section 4.3), written out: subtree sizes by a pass from the last
    node to the first, the heavy child of a node = its child with the largest subtree (lowest index on
    ties), and chains grown from their heads: a node continues its parent's chain iff it is the heavy
    child; children of the committed state head chains.  Returns (chain_head int32 [T], n_chains int32
    [B]): for every node the local index of the first node of its chain."""
    node_offsets, parent = _c(node_offsets, np.int32), _c(parent, np.int32)
    B = node_offsets.shape[0] - 1
    chain_head = np.zeros(parent.shape[0], np.int32)
    n_chains = np.zeros(B, np.int32)
    for b in range(B):
        base, n = int(node_offsets[b]), int(node_offsets[b + 1] - node_offsets[b])
        par = parent[base:base + n]
        size = [1] * n
        for t in range(n - 1, -1, -1):
            if par[t] >= 0:
                size[par[t]] += size[t]
        heavy = [-1] * n
        for t in range(n):                               # ascending: the first child of maximal size wins
            p = par[t]
            if p >= 0 and (heavy[p] < 0 or size[t] > size[heavy[p]]):
                heavy[p] = t
        for t in range(n):                               # parents come before children
            p = par[t]
            chain_head[base + t] = chain_head[base + p] if (p >= 0 and heavy[p] == t) else t
            n_chains[b] += int(chain_head[base + t] == t)
    return chain_head, n_chains
