"""Seeded synthetic inputs for the verify / accept / commit path.

This module holds NO arithmetic of the method: it only draws random arrays and
random tree topologies with the shapes, value ranges and structure of the
paper's GDN workloads (fp32 recurrent state, bf16 projected activations,
chains of up to 8 tokens and pruned draft trees of 16-64 nodes, Section 7 and
Section 8.1).  Both the CPU oracle's tests and the CUDA tests draw from it.

Arrays are numpy; q, k, v are stored as bf16 bit patterns in ``uint16``.

Draw order for a given seed: topology, S0, q, k, v, x_beta, x_alpha, token ids,
prescribed accepted paths.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np

VOCAB = 32000


# ----------------------------------------------------------------------------
# bf16 storage helpers (format conversion only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round to nearest even), return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# topologies
# ----------------------------------------------------------------------------
def chain_parent(n: int) -> np.ndarray:
    """parent[i] = i - 1: the chain special case p_j = j - 1 (Section 7)."""
    return np.arange(-1, n - 1, dtype=np.int32)


def depth_of(parent: np.ndarray) -> np.ndarray:
    """depth 1 for children of the committed state (the path sum of Section 6.1 starts at i = 1)."""
    d = np.zeros(len(parent), dtype=np.int32)
    for i, p in enumerate(parent):
        d[i] = 1 if p < 0 else d[p] + 1
    return d


def random_tree_parent(n: int, max_depth: int, max_children: int, rng: np.random.Generator) -> np.ndarray:
    """Single-rooted random tree in topological order.

    Node 0 hangs off the committed state; every later node picks its parent
    uniformly among earlier nodes that are shallower than ``max_depth`` and
    have fewer than ``max_children`` children.
    """
    parent = np.full(n, -1, dtype=np.int32)
    depth = np.ones(n, dtype=np.int32)
    nchild = np.zeros(n, dtype=np.int32)
    for i in range(1, n):
        ok = np.flatnonzero((depth[:i] < max_depth) & (nchild[:i] < max_children))
        if ok.size == 0:
            raise ValueError("no feasible parent: tree too large for max_depth/max_children")
        p = int(ok[rng.integers(ok.size)])
        parent[i] = p
        depth[i] = depth[p] + 1
        nchild[p] += 1
    return parent


def beam_tree_parent(top_k: int, depth: int, n_nodes: int, rng: np.random.Generator) -> np.ndarray:
    """EAGLE-style proposal shape: a per-level beam of ``top_k`` nodes down to
    ``depth`` levels, each level's nodes attached to random members of the
    previous level, truncated to ``n_nodes`` in level order (ancestor-closed)."""
    parent: List[int] = []
    prev: List[int] = [-1]
    level = 0
    while len(parent) < n_nodes and level < depth:
        cur: List[int] = []
        for j in range(top_k):
            if len(parent) >= n_nodes:
                break
            p = prev[0] if (level == 0 or j == 0) else prev[int(rng.integers(len(prev)))]
            parent.append(p)
            cur.append(len(parent) - 1)
        prev = cur
        level += 1
    return np.asarray(parent, dtype=np.int32)


def proposal_tree_parent(top_k: int, depth: int, n_nodes: int, rng: np.random.Generator,
                         max_depth: int = 16) -> np.ndarray:
    """Proposal tree with the metadata the paper reports per shape (top-k, configured depth,
    total nodes): ``n_nodes`` spread as evenly as possible over ``min(depth, max_depth)`` levels,
    a node having at most ``top_k`` children, parents drawn at random among the previous
    level's nodes that still have room.  Level order, so topological and ancestor-closed."""
    levels = min(depth, max_depth, n_nodes)
    width = [n_nodes // levels + (1 if i < n_nodes % levels else 0) for i in range(levels)]
    # a level can hold at most top_k children per node of the level above it
    cap = top_k
    for i in range(levels):
        if width[i] > cap:
            if i + 1 < levels:
                width[i + 1] += width[i] - cap
            width[i] = cap
        cap = width[i] * top_k
    parent: List[int] = []
    prev: List[int] = [-1]
    for w in width:
        room = {p: top_k for p in prev}
        cur: List[int] = []
        for j in range(w):
            cands = [p for p in prev if room[p] > 0]
            p = cands[0] if j == 0 else cands[int(rng.integers(len(cands)))]
            room[p] -= 1
            parent.append(p)
            cur.append(len(parent) - 1)
        prev = cur
    return np.asarray(parent, dtype=np.int32)


# ----------------------------------------------------------------------------
# problem container
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class Problem:
    L: int
    B: int
    H: int
    d_k: int
    d_v: int
    max_depth: int
    node_offsets: np.ndarray          # int32 [B+1]
    parent: np.ndarray                # int32 [T], local indices, -1 = committed state
    depth: np.ndarray                 # int32 [T]
    S0: np.ndarray                    # float32 [L,B,H,d_v,d_k]
    q: np.ndarray                     # uint16 (bf16) [L,T,H,d_k]
    k: np.ndarray                     # uint16 (bf16) [L,T,H,d_k]
    v: np.ndarray                     # uint16 (bf16) [L,T,H,d_v]
    alpha: np.ndarray                 # float32 [L,T,H]
    beta: np.ndarray                  # float32 [L,T,H]
    draft_tok: np.ndarray             # int32 [T]
    target_tok: np.ndarray            # int32 [T]
    root_target_tok: np.ndarray       # int32 [B]
    path_idx: Optional[np.ndarray] = None   # int32 [B,max_depth] prescribed accepted path (or None)
    path_len: Optional[np.ndarray] = None   # int32 [B]
    scale: float = 1.0
    name: str = ""

    @property
    def T(self) -> int:
        return int(self.node_offsets[-1])


def draw_state(rng, L, B, H, d_k, d_v, std=0.02) -> np.ndarray:
    return (rng.standard_normal((L, B, H, d_v, d_k), dtype=np.float32) * np.float32(std))


def draw_records(rng, L, T, H, d_k, d_v):
    """q, k, v ~ N(0,1) in fp32, k divided by its L2 norm in fp32, then all three
    rounded to bf16; beta = sigmoid(x_b), alpha = exp(-softplus(x_a)) = sigmoid(-x_a)
    evaluated in fp64 and cast to fp32."""
    q = rng.standard_normal((L, T, H, d_k), dtype=np.float32)
    k = rng.standard_normal((L, T, H, d_k), dtype=np.float32)
    k = k / np.sqrt(np.sum(k * k, axis=-1, keepdims=True, dtype=np.float32))
    v = rng.standard_normal((L, T, H, d_v), dtype=np.float32)
    xb = rng.standard_normal((L, T, H))
    xa = rng.standard_normal((L, T, H))
    beta = (1.0 / (1.0 + np.exp(-xb))).astype(np.float32)
    alpha = (1.0 / (1.0 + np.exp(xa))).astype(np.float32)
    return f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v), alpha, beta


def draw_tokens(rng, node_offsets: np.ndarray, parent: np.ndarray, p_match: float = 0.75):
    """Draft ids: siblings get distinct ids.  Target ids: for the committed state
    and every node with children, with probability ``p_match`` the target's greedy
    token equals one uniformly chosen child's draft id, else a uniform id; leaves
    get uniform ids."""
    B = len(node_offsets) - 1
    T = int(node_offsets[-1])
    draft = np.zeros(T, dtype=np.int32)
    target = np.zeros(T, dtype=np.int32)
    root_target = np.zeros(B, dtype=np.int32)
    for b in range(B):
        base, n = int(node_offsets[b]), int(node_offsets[b + 1] - node_offsets[b])
        children = {p: [] for p in range(-1, n)}
        for i in range(n):
            children[int(parent[base + i])].append(i)
        for p in range(-1, n):
            ch = children[p]
            if ch:
                ids = rng.choice(VOCAB, size=len(ch), replace=False)
                for c, t in zip(ch, ids):
                    draft[base + c] = t
        for p in range(-1, n):
            ch = children[p]
            if ch and rng.random() < p_match:
                tok = int(draft[base + ch[int(rng.integers(len(ch)))]])
            else:
                tok = int(rng.integers(VOCAB))
            if p < 0:
                root_target[b] = tok
            else:
                target[base + p] = tok
    return draft, target, root_target


def make_problem(seed: int, L: int, H: int, d_k: int, d_v: int, parents: Sequence[np.ndarray],
                 max_depth: int = 8, state_std: float = 0.02, p_match: float = 0.75,
                 name: str = "") -> Problem:
    """Assemble a packed batch from one parent array per sequence."""
    rng = np.random.default_rng(seed)
    return _assemble(rng, L, H, d_k, d_v, list(parents), max_depth, state_std, p_match, name)


def _assemble(rng, L, H, d_k, d_v, parents, max_depth, state_std, p_match, name) -> Problem:
    B = len(parents)
    sizes = [len(p) for p in parents]
    node_offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    parent = (np.concatenate(parents).astype(np.int32) if sum(sizes) else np.zeros(0, np.int32))
    depth = (np.concatenate([depth_of(p) for p in parents]).astype(np.int32)
             if sum(sizes) else np.zeros(0, np.int32))
    T = int(node_offsets[-1])
    S0 = draw_state(rng, L, B, H, d_k, d_v, state_std)
    q, k, v, alpha, beta = draw_records(rng, L, T, H, d_k, d_v)
    draft, target, root_target = draw_tokens(rng, node_offsets, parent, p_match)
    return Problem(L, B, H, d_k, d_v, max_depth, node_offsets, parent, depth, S0, q, k, v,
                   alpha, beta, draft, target, root_target, name=name)


def _set_paths(prob: Problem, paths: Sequence[Sequence[int]]) -> None:
    idx = np.full((prob.B, prob.max_depth), -1, dtype=np.int32)
    ln = np.zeros(prob.B, dtype=np.int32)
    for b, p in enumerate(paths):
        ln[b] = len(p)
        idx[b, :len(p)] = p
    prob.path_idx, prob.path_len = idx, ln


def root_path(parent: np.ndarray, node: int) -> List[int]:
    out = []
    a = int(node)
    while a >= 0:
        out.append(a)
        a = int(parent[a])
    return out[::-1]


def ragged_tree_batch(rng, B: int, n_lo: int, n_hi: int, max_depth: int, max_children: int = 4):
    return [random_tree_parent(int(rng.integers(n_lo, n_hi + 1)), max_depth, max_children, rng)
            for _ in range(B)]


def mixed_chain_tree_batch(rng, B: int, chain_len: int = 8, tree_nodes: int = 64, max_depth: int = 8):
    """First half of the batch: chains; second half: trees of ``tree_nodes`` nodes."""
    out = [chain_parent(chain_len) for _ in range(B // 2)]
    out += [random_tree_parent(tree_nodes, max_depth, 4, rng) for _ in range(B - B // 2)]
    return out


# ----------------------------------------------------------------------------
# the five benchmark configurations
# ----------------------------------------------------------------------------
def config(idx: int, seed: Optional[int] = None, *, L: Optional[int] = None,
           B: Optional[int] = None) -> Problem:
    """Workload ``idx`` (1-based).  ``L`` / ``B`` shrink the layer count or batch of
    the large configurations for tests; the default is the full size.

    1: 1 sequence, 1 layer, 4 heads, d=64, chain of 4, first 2 accepted, seed 0
    2: 1 sequence, 24 layers, 16 heads, d=128, chain of 8, accepted length U{0..8}
    3: same dims, 32-node tree, depth <= 6, <= 4 children, random root-to-leaf path accepted
    4: 32 sequences, 24 layers, 16 heads, d_k=128, d_v=256, ragged trees of 8..64 nodes, depth <= 8
    5: 128 sequences, same dims, half 8-chains and half 64-node trees
    """
    if seed is None:
        seed = 0 if idx == 1 else 1000 + idx
    rng = np.random.default_rng(seed)
    if idx == 1:
        prob = _assemble(rng, L or 1, 4, 64, 64, [chain_parent(4)], 8, 0.02, 0.75, "cfg1")
        _set_paths(prob, [[0, 1]])
    elif idx == 2:
        prob = _assemble(rng, L or 24, 16, 128, 128, [chain_parent(8)], 8, 0.02, 0.75, "cfg2")
        a = int(rng.integers(0, 9))
        _set_paths(prob, [list(range(a))])
    elif idx == 3:
        par = random_tree_parent(32, 6, 4, rng)
        prob = _assemble(rng, L or 24, 16, 128, 128, [par], 8, 0.02, 0.75, "cfg3")
        has_child = np.zeros(32, dtype=bool)
        has_child[par[par >= 0]] = True
        leaves = np.flatnonzero(~has_child)
        leaf = int(leaves[rng.integers(leaves.size)])
        _set_paths(prob, [root_path(par, leaf)])
    elif idx == 4:
        parents = ragged_tree_batch(rng, B or 32, 8, 64, 8)
        prob = _assemble(rng, L or 24, 16, 128, 256, parents, 8, 0.02, 0.75, "cfg4")
    elif idx == 5:
        parents = mixed_chain_tree_batch(rng, B or 128, 8, 64, 8)
        prob = _assemble(rng, L or 24, 16, 128, 256, parents, 8, 0.02, 0.75, "cfg5")
    else:
        raise ValueError("config index must be 1..5")
    return prob


def gather_units(prob: Problem, units: Sequence[tuple]) -> Problem:
    """Copy the listed (layer, sequence, head) units into a small problem with
    L=1, H=1 and one sequence per listed unit (units are independent, so this is
    pure re-packing).  Used to check a sample of a large workload."""
    parents, S0, q, k, v, al, be = [], [], [], [], [], [], []
    for (l, b, h) in units:
        s, e = int(prob.node_offsets[b]), int(prob.node_offsets[b + 1])
        parents.append(prob.parent[s:e].copy())
        S0.append(prob.S0[l, b, h])
        q.append(prob.q[l, s:e, h]); k.append(prob.k[l, s:e, h]); v.append(prob.v[l, s:e, h])
        al.append(prob.alpha[l, s:e, h]); be.append(prob.beta[l, s:e, h])
    sizes = [len(p) for p in parents]
    node_offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    sub = Problem(
        1, len(units), 1, prob.d_k, prob.d_v, prob.max_depth, node_offsets,
        np.concatenate(parents).astype(np.int32),
        np.concatenate([depth_of(p) for p in parents]).astype(np.int32),
        np.stack(S0)[None, :, None], np.concatenate(q)[None, :, None], np.concatenate(k)[None, :, None],
        np.concatenate(v)[None, :, None], np.concatenate(al)[None, :, None], np.concatenate(be)[None, :, None],
        np.zeros(int(node_offsets[-1]), np.int32), np.zeros(int(node_offsets[-1]), np.int32),
        np.zeros(len(units), np.int32), scale=prob.scale, name=prob.name + "/sample")
    if prob.path_idx is not None:
        sub.path_idx = np.stack([prob.path_idx[b] for (_, b, _) in units]).astype(np.int32)
        sub.path_len = np.asarray([prob.path_len[b] for (_, b, _) in units], dtype=np.int32)
    return sub


# ----------------------------------------------------------------------------
# on-device drawing for the multi-GB configurations (same distributions, torch RNG)
# ----------------------------------------------------------------------------
def device_state(seed: int, L: int, B: int, H: int, d_k: int, d_v: int, std: float = 0.02, device="cuda"):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    S = torch.empty((L, B, H, d_v, d_k), dtype=torch.float32, device=device)
    for l in range(L):                       # layer by layer: no multi-GB temporaries
        S[l].normal_(0.0, std, generator=g)
    return S


def device_records(seed: int, L: int, T: int, H: int, d_k: int, d_v: int, device="cuda"):
    """q, k, v (bf16), alpha, beta (fp32) with the distributions of ``draw_records``."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    q = torch.empty((L, T, H, d_k), dtype=torch.bfloat16, device=device)
    k = torch.empty((L, T, H, d_k), dtype=torch.bfloat16, device=device)
    v = torch.empty((L, T, H, d_v), dtype=torch.bfloat16, device=device)
    for l in range(L):
        q[l] = torch.randn((T, H, d_k), generator=g, device=device)
        kk = torch.randn((T, H, d_k), generator=g, device=device)
        k[l] = kk / kk.norm(dim=-1, keepdim=True)
        v[l] = torch.randn((T, H, d_v), generator=g, device=device)
    xb = torch.randn((L, T, H), generator=g, device=device, dtype=torch.float64)
    xa = torch.randn((L, T, H), generator=g, device=device, dtype=torch.float64)
    beta = torch.sigmoid(xb).float()
    alpha = torch.sigmoid(-xa).float()
    return q, k, v, alpha, beta
