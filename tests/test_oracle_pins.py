"""Pins for the fp64 oracle: what the mathematics and the paper fix, computed by
routes that share nothing with oracle/gdn_oracle.c.

  * hand-worked scalar cases and closed forms of the gated delta rule
  * a dense-matrix restatement (transition matrix built explicitly, numpy matmul)
  * the tree-masked UT/WY factorisation of Section 4.2, solved densely
  * snapshot propagation over EVERY forest of <= 4 nodes
  * structural invariants: chain == repeated decode, single-path tree == chain,
    commit == sequential recurrence, sibling isolation, linearity in (S0, V),
    row independence, relabelling by another topological order
  * acceptance: brute force over all root paths, hand cases; the stochastic rule: hand cases, min(1, p/q),
    the closed-form length distribution on chains, a level-free restatement
  * heavy-light chains: the chains the paper prints for its example, partition / path / log-bound properties
  * byte counts printed by the paper (state, snapshots, factor buffer)
"""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2607_16673_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------
# independent numpy formulations
# ---------------------------------------------------------------------------
def dense_rule(S, k, v, a, b):
    """S * alpha (I - beta k k^T) + beta v k^T with the d_k x d_k transition matrix formed explicitly."""
    dk = k.shape[0]
    return S @ (a * (np.eye(dk) - b * np.outer(k, k))) + b * np.outer(v, k)


def snapshot_verify(S0, q, k, v, al, be, parent):
    """Keep one dense state per node (the 'full-state snapshot' strategy of Section 5.1)."""
    n = len(parent)
    states, outs = [None] * n, []
    for t in range(n):
        Sp = S0 if parent[t] < 0 else states[parent[t]]
        states[t] = dense_rule(Sp, k[t], v[t], al[t], be[t])
        outs.append(states[t] @ q[t])
    return np.array(outs).reshape(n, S0.shape[0]), states


def factorised_verify(S0, q, k, v, al, be, parent):
    """Tree-masked factorised form (Section 4.2): A_tree = M_tree o (K_b K_a^T),
    T = (I - A_tree)^-1, O = Qhat S0^T - Attn (W S0^T) + Attn U."""
    n = len(parent)
    gamma = np.zeros(n)
    anc = np.zeros((n, n), dtype=bool)            # strict ancestor mask (M_tree without the diagonal)
    for t in range(n):
        p = parent[t]
        gamma[t] = al[t] * (1.0 if p < 0 else gamma[p])
        if p >= 0:
            anc[t] = anc[p]
            anc[t, p] = True
    Ka = k / gamma[:, None]
    Kb = -(be * gamma)[:, None] * k
    A = np.where(anc, Kb @ Ka.T, 0.0)
    Tm = np.linalg.inv(np.eye(n) - A)
    W = Tm @ ((be * gamma)[:, None] * k)
    Ut = Tm @ (be[:, None] * v)
    Qh = gamma[:, None] * q
    Attn = np.where(anc | np.eye(n, dtype=bool), Qh @ Ka.T, 0.0)
    return Qh @ S0.T - Attn @ (W @ S0.T) + Attn @ Ut


def unit_arrays(prob, l=0, b=0, h=0):
    s, e = int(prob.node_offsets[b]), int(prob.node_offsets[b + 1])
    f = lambda a: synth.bf16_bits_to_f32(a[l, s:e, h]).astype(np.float64)
    return (prob.S0[l, b, h].astype(np.float64), f(prob.q), f(prob.k), f(prob.v),
            prob.alpha[l, s:e, h].astype(np.float64), prob.beta[l, s:e, h].astype(np.float64),
            prob.parent[s:e])


def run_verify(prob, **over):
    g = lambda name: over.get(name, getattr(prob, name))
    return oracle.verify_tree(g("S0"), g("q"), g("k"), g("v"), g("alpha"), g("beta"),
                              g("node_offsets"), g("parent"), prob.scale)


def bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def one_token(S0, q, k, v, a, b):
    """Oracle decode of one unit given float arrays (exactly representable in bf16)."""
    dv, dk = S0.shape
    S, o = oracle.decode_step(S0[None, None, None], bits(q)[None, None, None], bits(k)[None, None, None],
                              bits(v)[None, None, None], np.full((1, 1, 1), a, np.float32),
                              np.full((1, 1, 1), b, np.float32))
    return S[0, 0, 0], o[0, 0, 0]


# ---------------------------------------------------------------------------
# hand-worked values and closed forms
# ---------------------------------------------------------------------------
def test_hand_worked_scalar_cases():
    """tests/golden/gdn_scalar_cases.txt: 1x1 states worked by hand from the rule."""
    rows = [r.split() for r in open(os.path.join(GOLDEN, "gdn_scalar_cases.txt"))
            if r.strip() and not r.startswith("#")]
    assert len(rows) >= 4
    for r in rows:
        S, k, v, a, b, q, S1, o = map(float, r)
        Sn, on = one_token(np.array([[S]]), [q], [k], [v], a, b)
        assert Sn[0, 0] == pytest.approx(S1, rel=1e-15, abs=1e-15)
        assert on[0] == pytest.approx(o, rel=1e-15, abs=1e-15)


def test_hand_worked_2x2_case():
    """S=[[1,2],[3,4]], k=(1,0), v=(5,6), alpha=0.5, beta=0.5, q=(1,1):
    decayed = [[.5,1],[1.5,2]]; read = (.5,1.5); S' = decayed + .5*(v-read) k^T
            = [[.5+2.25, 1],[1.5+2.25, 2]] = [[2.75,1],[3.75,2]]; o = (3.75, 5.75)."""
    Sn, on = one_token(np.array([[1., 2.], [3., 4.]]), [1, 1], [1, 0], [5, 6], 0.5, 0.5)
    assert np.array_equal(Sn, np.array([[2.75, 1.0], [3.75, 2.0]]))
    assert np.array_equal(on, np.array([3.75, 5.75]))


def test_zero_state_single_token_is_outer_product():
    rng = np.random.default_rng(1)
    dk, dv = 16, 8
    q, k, v, al, be = synth.draw_records(rng, 1, 1, 1, dk, dv)
    S, o = oracle.decode_step(np.zeros((1, 1, 1, dv, dk)), q, k, v, al, be)
    kf, vf, qf = (synth.bf16_bits_to_f32(x).astype(np.float64).ravel() for x in (k, v, q))
    b = float(be.ravel()[0])
    assert np.allclose(S[0, 0, 0], b * np.outer(vf, kf), rtol=1e-15, atol=0)
    assert np.allclose(o[0, 0, 0], b * vf * (kf @ qf), rtol=1e-13, atol=1e-15)


def test_delta_rule_retrieval_unit_key():
    """alpha = beta = 1 and |k| = 1  =>  S_1 k = v exactly (the delta rule overwrites the slot)."""
    rng = np.random.default_rng(2)
    dk, dv = 64, 32
    k = rng.choice([-1.0, 1.0], size=dk) / 8.0            # exact in bf16, norm exactly 1
    v = synth.bf16_bits_to_f32(bits(rng.standard_normal(dv))).astype(np.float64)
    S0 = rng.standard_normal((dv, dk))
    S1, _ = one_token(S0, np.zeros(dk), k, v, 1.0, 1.0)
    assert np.allclose(S1 @ k, v, rtol=0, atol=1e-13)
    # directions orthogonal to k are untouched
    w = np.zeros(dk); w[0], w[1] = k[1], -k[0]
    assert np.allclose(S1 @ w, S0 @ w, rtol=0, atol=1e-13)


def test_read_after_write_identity_general():
    """S_t k_t = alpha (1 - beta |k|^2) S_{t-1} k_t + beta |k|^2 v_t."""
    rng = np.random.default_rng(3)
    dk, dv = 32, 16
    q, k, v, al, be = synth.draw_records(rng, 1, 1, 1, dk, dv)
    S0 = rng.standard_normal((1, 1, 1, dv, dk))
    S1, _ = oracle.decode_step(S0, q, k, v, al, be)
    kf = synth.bf16_bits_to_f32(k).astype(np.float64).ravel()
    vf = synth.bf16_bits_to_f32(v).astype(np.float64).ravel()
    a, b, n2 = float(al.ravel()[0]), float(be.ravel()[0]), float(kf @ kf)
    assert np.allclose(S1[0, 0, 0] @ kf, a * (1 - b * n2) * (S0[0, 0, 0] @ kf) + b * n2 * vf,
                       rtol=1e-12, atol=1e-13)


def test_orthonormal_keys_reduce_to_linear_attention():
    """alpha = beta = 1, S_0 = 0, orthonormal keys: S_n = sum v_i k_i^T (Eq. 1) and
    o_n = sum_i v_i (k_i . q_n) -- causal linear attention."""
    rng = np.random.default_rng(4)
    dk, dv, n = 16, 8, 6
    K = np.eye(dk)[:n]
    V = synth.bf16_bits_to_f32(bits(rng.standard_normal((n, dv)))).astype(np.float64)
    Q = synth.bf16_bits_to_f32(bits(rng.standard_normal((n, dk)))).astype(np.float64)
    offs = np.array([0, n], np.int32)
    ones = np.ones((1, n, 1), np.float32)
    o = oracle.verify_chain(np.zeros((1, 1, 1, dv, dk)), bits(Q)[None, :, None], bits(K)[None, :, None],
                            bits(V)[None, :, None], ones, ones, offs)[0, :, 0]
    expect = np.tril(Q @ K.T) @ V
    assert np.allclose(o, expect, rtol=0, atol=1e-14)
    path_idx = np.arange(8, dtype=np.int32)[None]
    S = oracle.commit(np.zeros((1, 1, 1, dv, dk)), bits(K)[None, :, None], bits(V)[None, :, None], ones, ones,
                      offs, path_idx, np.array([n], np.int32))
    assert np.allclose(S[0, 0, 0], V.T @ K, rtol=0, atol=1e-14)


def test_beta_zero_is_pure_decay_and_alpha_one_is_identity():
    prob = synth.make_problem(5, 2, 2, 16, 8, [synth.random_tree_parent(7, 4, 3, np.random.default_rng(5))])
    zero = np.zeros_like(prob.beta)
    o = run_verify(prob, beta=zero)
    S0, q, k, v, al, be, par = unit_arrays(prob, 1, 0, 1)
    for t in range(len(par)):
        g = np.prod([al[a] for a in synth.root_path(par, t)])
        assert np.allclose(o[1, t, 1], g * (S0 @ q[t]), rtol=1e-13, atol=1e-15)
    one = np.ones_like(prob.alpha)
    o1 = run_verify(prob, beta=zero, alpha=one)
    assert np.allclose(o1[1, :, 1], q @ S0.T, rtol=1e-13, atol=1e-15)
    path = np.full((1, 8), -1, np.int32); path[0, :3] = synth.root_path(par, 6)[:3]
    n_acc = min(3, len(synth.root_path(par, 6)))
    Sc = oracle.commit(prob.S0, prob.k, prob.v, one, zero, prob.node_offsets, path, np.array([n_acc], np.int32))
    assert np.array_equal(Sc, prob.S0.astype(np.float64))


# ---------------------------------------------------------------------------
# independent formulations
# ---------------------------------------------------------------------------
def test_decode_matches_dense_matrix_form():
    rng = np.random.default_rng(6)
    L, B, H, dk, dv = 2, 3, 2, 24, 12
    S0 = rng.standard_normal((L, B, H, dv, dk))
    q, k, v, al, be = synth.draw_records(rng, L, B, H, dk, dv)
    S1, o = oracle.decode_step(S0, q, k, v, al, be, scale=0.5)
    f = lambda a: synth.bf16_bits_to_f32(a).astype(np.float64)
    for l, b, h in itertools.product(range(L), range(B), range(H)):
        ref = dense_rule(S0[l, b, h], f(k)[l, b, h], f(v)[l, b, h], float(al[l, b, h]), float(be[l, b, h]))
        assert np.allclose(S1[l, b, h], ref, rtol=1e-12, atol=1e-14)
        assert np.allclose(o[l, b, h], 0.5 * ref @ f(q)[l, b, h], rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("seed,n,max_depth", [(7, 12, 5), (8, 24, 6), (9, 40, 8)])
def test_verify_matches_tree_masked_factorisation(seed, n, max_depth):
    par = synth.random_tree_parent(n, max_depth, 4, np.random.default_rng(seed))
    prob = synth.make_problem(seed, 1, 2, 32, 16, [par], state_std=0.5)
    o = run_verify(prob)
    for h in range(2):
        S0, q, k, v, al, be, p = unit_arrays(prob, 0, 0, h)
        ref = factorised_verify(S0, q, k, v, al, be, p)
        assert np.allclose(o[0, :, h], ref, rtol=1e-9, atol=1e-10)


def all_forests(n):
    return itertools.product(*[range(-1, i) for i in range(n)])


def test_brute_force_all_forests_up_to_4_nodes():
    count = 0
    for n in range(1, 5):
        for par in all_forests(n):
            par = np.array(par, np.int32)
            prob = synth.make_problem(100 + count, 1, 1, 8, 4, [par], state_std=1.0)
            o = run_verify(prob)[0, :, 0]
            S0, q, k, v, al, be, p = unit_arrays(prob)
            ref, states = snapshot_verify(S0, q, k, v, al, be, p)
            assert np.allclose(o, ref, rtol=1e-12, atol=1e-13), par
            # commit along every root path reproduces that node's snapshot
            for t in range(n):
                path = synth.root_path(par, t)
                idx = np.full((1, 8), -1, np.int32); idx[0, :len(path)] = path
                Sc = oracle.commit(prob.S0, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets,
                                   idx, np.array([len(path)], np.int32))
                assert np.allclose(Sc[0, 0, 0], states[t], rtol=1e-12, atol=1e-13)
            count += 1
    assert count == 1 + 2 + 6 + 24


# ---------------------------------------------------------------------------
# structural invariants
# ---------------------------------------------------------------------------
def test_chain_verify_equals_repeated_decode_and_commit():
    prob = synth.config(1)
    n = prob.T
    o = oracle.verify_chain(prob.S0, prob.q, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets)
    S = prob.S0.astype(np.float64)
    for t in range(n):
        S, ot = oracle.decode_step(S, prob.q[:, t:t + 1], prob.k[:, t:t + 1], prob.v[:, t:t + 1],
                                   prob.alpha[:, t:t + 1], prob.beta[:, t:t + 1])
        assert np.array_equal(ot[:, 0], o[:, t])          # same arithmetic, same order: bit-identical
        idx = np.full((1, 8), -1, np.int32); idx[0, :t + 1] = np.arange(t + 1)
        Sc = oracle.commit(prob.S0, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets,
                           idx, np.array([t + 1], np.int32))
        assert np.array_equal(Sc, S)
    # accepted length 0 leaves the state untouched
    S_same = oracle.commit(prob.S0, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets,
                           np.full((1, 8), -1, np.int32), np.zeros(1, np.int32))
    assert np.array_equal(S_same, prob.S0.astype(np.float64))


def test_single_path_tree_equals_chain():
    prob = synth.make_problem(11, 2, 2, 16, 16, [synth.chain_parent(6), synth.chain_parent(3)])
    a = run_verify(prob)
    b = oracle.verify_chain(prob.S0, prob.q, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets)
    assert np.array_equal(a, b)


def test_root_to_leaf_replay_equals_tree_verify():
    """Verifying each root path as its own chain (the replay baseline of Section 4.2) gives the same outputs."""
    par = synth.random_tree_parent(14, 5, 3, np.random.default_rng(12))
    prob = synth.make_problem(12, 1, 2, 16, 8, [par])
    o = run_verify(prob)
    for t in range(14):
        path = synth.root_path(par, t)
        sel = np.array(path)
        oc = oracle.verify_chain(prob.S0, prob.q[:, sel], prob.k[:, sel], prob.v[:, sel], prob.alpha[:, sel],
                                 prob.beta[:, sel], np.array([0, len(path)], np.int32))
        assert np.array_equal(oc[:, -1], o[:, t])


def test_delayed_update_identities():
    """What the fused commit-and-verify relies on (Section 5.2, Eq. 3):
    (1) committing an accepted path and verifying a new draft from the committed state equals verifying
        the tree obtained by hanging the new draft under the last accepted node, restricted to the new nodes;
    (2) the committed state is gamma_A S0 + sum_i (gamma_A / gamma_i) u_i k_i^T, with u_i = beta_i (v_i - alpha_i S_{i-1} k_i)
        the corrected values of the accepted nodes -- checked here with numpy only from the dense rule."""
    rng = np.random.default_rng(31)
    par1 = synth.random_tree_parent(11, 5, 3, rng)
    par2 = synth.random_tree_parent(9, 4, 3, rng)
    p1 = synth.make_problem(31, 2, 2, 16, 8, [par1])
    p2 = synth.make_problem(32, 2, 2, 16, 8, [par2])
    path = synth.root_path(par1, 10)
    A = len(path)
    idx = np.full((1, 8), -1, np.int32); idx[0, :A] = path
    S1 = oracle.commit(p1.S0, p1.k, p1.v, p1.alpha, p1.beta, p1.node_offsets, idx, np.array([A], np.int32))
    o_new = oracle.verify_tree(S1, p2.q, p2.k, p2.v, p2.alpha, p2.beta, p2.node_offsets, p2.parent)
    # (1) spliced tree: accepted path as a chain, then the new nodes with their roots under its last node
    sel = np.array(path)
    cat = lambda a, b: np.concatenate([a[:, sel], b], axis=1)
    par_sp = np.concatenate([np.arange(-1, A - 1), np.where(par2 < 0, A - 1, par2 + A)]).astype(np.int32)
    o_sp = oracle.verify_tree(p1.S0, cat(p1.q, p2.q), cat(p1.k, p2.k), cat(p1.v, p2.v), cat(p1.alpha, p2.alpha),
                              cat(p1.beta, p2.beta), np.array([0, A + len(par2)], np.int32), par_sp)
    assert np.allclose(o_sp[:, A:], o_new, rtol=1e-12, atol=1e-14)
    # (2) rank-A form of the committed state, unit (layer 1, head 0)
    S0, q, k, v, al, be, _ = unit_arrays(p1, l=1, b=0, h=0)
    S, us, gam = S0.copy(), [], []
    g = 1.0
    for t in path:
        us.append(be[t] * (v[t] - al[t] * (S @ k[t])))
        S = dense_rule(S, k[t], v[t], al[t], be[t])
        g *= al[t]
        gam.append(g)
    S_rank = g * S0 + sum((g / gam[i]) * np.outer(us[i], k[t]) for i, t in enumerate(path))
    assert np.allclose(S_rank, S, rtol=1e-12, atol=1e-14)
    assert np.allclose(S1[1, 0, 0], S, rtol=1e-12, atol=1e-14)


def test_sibling_isolation():
    """Changing any factor of node t changes outputs of t and its descendants only (tree mask, Section 4.2)."""
    rng = np.random.default_rng(13)
    par = synth.random_tree_parent(16, 5, 3, rng)
    prob = synth.make_problem(13, 1, 1, 16, 8, [par])
    base = run_verify(prob)
    for t in [0, 3, 7, 15]:
        desc = np.array([t in synth.root_path(par, j) for j in range(16)])
        for name in ["k", "v", "alpha", "beta"]:
            arr = getattr(prob, name).copy()
            if arr.dtype == np.uint16:
                arr[0, t, 0] = bits(synth.bf16_bits_to_f32(arr[0, t, 0]) * 1.5 + 0.25)
            else:
                arr[0, t, 0] = 0.5 * arr[0, t, 0] + 0.1
            o = run_verify(prob, **{name: arr})
            changed = np.any(o[0, :, 0] != base[0, :, 0], axis=-1)
            assert np.array_equal(changed, desc), (t, name)
        arr = prob.q.copy(); arr[0, t, 0] = bits(synth.bf16_bits_to_f32(arr[0, t, 0]) + 1.0)
        changed = np.any(run_verify(prob, q=arr)[0, :, 0] != base[0, :, 0], axis=-1)
        assert np.array_equal(changed, np.arange(16) == t)


def test_joint_linearity_in_state_and_values():
    par = synth.random_tree_parent(10, 4, 3, np.random.default_rng(14))
    prob = synth.make_problem(14, 1, 2, 16, 8, [par], state_std=1.0)
    full = run_verify(prob)
    only_state = run_verify(prob, v=np.zeros_like(prob.v))
    only_values = run_verify(prob, S0=np.zeros_like(prob.S0))
    assert np.allclose(full, only_state + only_values, rtol=1e-12, atol=1e-13)


def test_row_independence():
    """Rows of S are independent recurrences (the V-tiling argument, Section 4.1)."""
    par = synth.random_tree_parent(9, 4, 3, np.random.default_rng(15))
    prob = synth.make_problem(15, 1, 1, 16, 8, [par], state_std=1.0)
    perm = np.random.default_rng(15).permutation(8)
    o = run_verify(prob)
    op = run_verify(prob, S0=prob.S0[..., perm, :], v=prob.v[..., perm])
    assert np.array_equal(op, o[..., perm])


def test_relabelling_by_another_topological_order():
    rng = np.random.default_rng(16)
    par = synth.random_tree_parent(12, 5, 3, rng)
    prob = synth.make_problem(16, 1, 1, 16, 8, [par])
    o = run_verify(prob)
    # DFS preorder is another topological order
    children = {i: [j for j in range(12) if par[j] == i] for i in range(-1, 12)}
    order, stack = [], list(reversed(children[-1]))
    while stack:
        x = stack.pop(); order.append(x); stack.extend(reversed(children[x]))
    order = np.array(order); inv = np.empty(12, int); inv[order] = np.arange(12)
    par2 = np.array([-1 if par[x] < 0 else inv[par[x]] for x in order], np.int32)
    o2 = run_verify(prob, parent=par2, q=prob.q[:, order], k=prob.k[:, order], v=prob.v[:, order],
                    alpha=prob.alpha[:, order], beta=prob.beta[:, order])
    assert np.array_equal(o2, o[:, order])


def test_scale_multiplies_outputs():
    prob = synth.config(1)
    o1 = run_verify(prob)
    prob.scale = 0.25
    assert np.array_equal(run_verify(prob), 0.25 * o1)


# ---------------------------------------------------------------------------
# greedy acceptance
# ---------------------------------------------------------------------------
def brute_accept(parent, draft, target, root_target, max_depth):
    """Enumerate every root path; keep those whose every token equals the prediction made at its parent."""
    n = len(parent)
    best = []
    for t in range(n):
        path = synth.root_path(parent, t)
        ok = all(draft[a] == (root_target if parent[a] < 0 else target[parent[a]]) for a in path)
        if ok and len(path) > len(best):
            best = path
    nxt = root_target if not best else target[best[-1]]
    return best, nxt


def accept_one(parent, draft, target, root_target, max_depth=8):
    parent = np.asarray(parent, np.int32)
    offs = np.array([0, len(parent)], np.int32)
    pi, pl, nt = oracle.greedy_accept(offs, parent, np.asarray(draft, np.int32), np.asarray(target, np.int32),
                                      np.array([root_target], np.int32), max_depth)
    return list(pi[0, :pl[0]]), int(pl[0]), int(nt[0]), pi[0]


def test_accept_hand_cases():
    # chain 0-1-2, all match
    assert accept_one([-1, 0, 1], [5, 6, 7], [6, 7, 8], 5)[:3] == ([0, 1, 2], 3, 8)
    # no match at the root: empty path, next token is the root prediction
    path, ln, nxt, raw = accept_one([-1, 0, 1], [5, 6, 7], [6, 7, 8], 9)
    assert (path, ln, nxt) == ([], 0, 9) and np.all(raw == -1)
    # match stops at an internal node
    assert accept_one([-1, 0, 1], [5, 6, 7], [6, 1, 8], 5)[:3] == ([0, 1], 2, 1)
    # the accepted sibling is not the first one; deeper descendant of an unmatched sibling is ignored
    #      -1 -> 0(tok 3), 1(tok 4);  0 -> 2(tok 9);  1 -> 3(tok 8)
    assert accept_one([-1, -1, 0, 1], [3, 4, 9, 8], [9, 8, 0, 11], 4)[:3] == ([1, 3], 2, 11)
    # a descendant that matches its own parent's prediction does not count when the parent is unmatched
    assert accept_one([-1, 0], [3, 9], [9, 1], 4)[:3] == ([], 0, 4)


def test_accept_matches_brute_force_on_random_trees():
    rng = np.random.default_rng(17)
    lengths = []
    for trial in range(200):
        n = int(rng.integers(1, 20))
        par = synth.random_tree_parent(n, 8, 4, rng)
        offs = np.array([0, n], np.int32)
        draft, target, root = synth.draw_tokens(rng, offs, par, p_match=0.8)
        path, ln, nxt, _ = accept_one(par, draft, target, int(root[0]))
        bpath, bnxt = brute_accept(par, draft, target, int(root[0]), 8)
        assert path == bpath and nxt == bnxt
        lengths.append(ln)
    assert max(lengths) >= 3 and min(lengths) == 0


def test_accept_batched_offsets():
    rng = np.random.default_rng(18)
    parents = synth.ragged_tree_batch(rng, 6, 1, 12, 5)
    prob = synth.make_problem(18, 1, 1, 8, 8, parents)
    pi, pl, nt = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                      prob.root_target_tok, 8)
    for b in range(6):
        s, e = prob.node_offsets[b], prob.node_offsets[b + 1]
        bpath, bnxt = brute_accept(prob.parent[s:e], prob.draft_tok[s:e], prob.target_tok[s:e],
                                   int(prob.root_target_tok[b]), 8)
        assert list(pi[b, :pl[b]]) == bpath and nt[b] == bnxt


# ---------------------------------------------------------------------------
# sizes the paper prints (pin the layouts and the record contents)
# ---------------------------------------------------------------------------
def test_conv_state_commit_hand_cases_and_convolution_identity():
    """The convolution state is a shift register of the last W inputs (kernel size W + 1).  Hand cases,
    and the property that defines it: the next token's causal convolution output computed from the
    committed register equals the direct convolution (numpy.convolve) over the whole input history."""
    u16 = lambda *v: np.array(v, np.uint16)
    C = u16(1, 2, 3).reshape(1, 1, 3, 1)
    x = u16(10, 11, 12, 13, 14).reshape(1, 5, 1)
    offs = np.array([0, 5], np.int32)
    idx = lambda *p: np.array([list(p) + [-1] * (8 - len(p))], np.int32)
    run = lambda p: oracle.commit_conv(C, x, offs, idx(*p), np.array([len(p)], np.int32))[0, 0, :, 0].tolist()
    assert run([]) == [1, 2, 3]
    assert run([0]) == [2, 3, 10]
    assert run([0, 2]) == [3, 10, 12]
    assert run([0, 2, 3]) == [10, 12, 13]
    assert run([0, 1, 2, 4]) == [11, 12, 14]
    # convolution identity on random data: 2 layers, 3 sequences, kernel size 4, 5 channels
    rng = np.random.default_rng(41)
    L, B, W, ch = 2, 3, 3, 5
    parents = [synth.random_tree_parent(9, 5, 3, rng), synth.chain_parent(2), synth.random_tree_parent(6, 6, 2, rng)]
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    T = int(offs[-1])
    hist = rng.standard_normal((L, B, 7, ch)).astype(np.float32)                # inputs seen before the draft
    Cb = synth.f32_to_bf16_bits(hist[:, :, -W:])
    xb = synth.f32_to_bf16_bits(rng.standard_normal((L, T, ch)).astype(np.float32))
    paths = [synth.root_path(parents[0], 8), [], synth.root_path(parents[2], 5)]
    pidx = np.full((B, 8), -1, np.int32); plen = np.zeros(B, np.int32)
    for b, pth in enumerate(paths):
        pidx[b, :len(pth)] = pth; plen[b] = len(pth)
    Cn = oracle.commit_conv(Cb, xb, offs, pidx, plen)
    wts = rng.standard_normal((ch, W + 1))                                      # taps, newest input last
    nxt = rng.standard_normal((L, B, ch))                                       # the next token's input
    f = lambda bits: synth.bf16_bits_to_f32(bits).astype(np.float64)
    for l in range(L):
        for b in range(B):
            seq = np.concatenate([f(synth.f32_to_bf16_bits(hist[l, b])), f(xb[l, offs[b] + np.array(paths[b], int)]).reshape(-1, ch),
                                  nxt[l, b][None]], axis=0)
            for c in range(ch):
                direct = np.convolve(seq[:, c], wts[c, ::-1])[len(seq) - 1]         # causal output at the last position
                from_state = np.dot(wts[c, :W], f(Cn[l, b, :, c])) + wts[c, W] * nxt[l, b, c]
                assert abs(direct - from_state) <= 1e-12 * (1 + abs(direct))
    assert np.array_equal(Cn[:, 1], Cb[:, 1])                                   # nothing accepted: untouched


def _mask_of(parents, N):
    """Tree attention mask built by walking every root path (independent of the converter)."""
    m = np.zeros((len(parents), N, N), np.uint8)
    for b, par in enumerate(parents):
        for i in range(len(par)):
            for a in synth.root_path(par, i):
                m[b, i, a] = 1
    return m


def test_tree_mask_converter_round_trip():
    rng = np.random.default_rng(51)
    parents = [synth.random_tree_parent(int(rng.integers(1, 30)), 8, 4, rng) for _ in range(6)]
    parents += [np.array([-1, -1, 0, -1, 1], np.int32), np.zeros(0, np.int32), synth.chain_parent(7)]
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    got = oracle.tree_mask_to_parent(_mask_of(parents, 32), offs)
    assert np.array_equal(got, np.concatenate(parents))


def test_pruning_hand_case_and_selection_properties():
    """Section 6.1: window q >= q* - tau on cumulative log-probabilities, then the budget."""
    #        0(-0.5)            3(-2.0)
    #       /      \
    #   1(-0.25)  2(-1.0)            q: 0:-0.5  1:-0.75  2:-1.5  3:-2.0  4:-0.875 (child of 1, -0.125)
    par = np.array([-1, 0, 0, -1, 1], np.int32)
    lp = np.array([-0.5, -0.25, -1.0, -2.0, -0.125], np.float32)
    offs = np.array([0, 5], np.int32)
    keep = lambda tau, T: oracle.prune_tree(offs, par, lp, tau, T)
    o, p, idx = keep(0.4, 8)                          # window: q >= -0.9 -> nodes 0, 1, 4
    assert idx.tolist() == [0, 1, 4] and p.tolist() == [-1, 0, 1] and o.tolist() == [0, 3]
    assert keep(1.0, 8)[2].tolist() == [0, 1, 2, 4]   # q >= -1.5
    assert keep(5.0, 8)[2].tolist() == [0, 1, 2, 3, 4]
    assert keep(5.0, 2)[2].tolist() == [0, 1]         # budget cuts the score-ranked selection
    assert keep(0.0, 8)[2].tolist() == [0]            # only q*
    assert keep(5.0, 0)[2].tolist() == []
    # properties on random trees with scores that are exact in fp32 (multiples of 1/8): the kept set is the
    # top-`budget` of the window by (q, index) computed independently in float64 with Python's sort
    rng = np.random.default_rng(52)
    parents = [synth.random_tree_parent(int(rng.integers(1, 40)), 8, 4, rng) for _ in range(8)]
    offs = np.concatenate([[0], np.cumsum([len(pp) for pp in parents])]).astype(np.int32)
    parent = np.concatenate(parents)
    logp = (-rng.integers(0, 12, int(offs[-1])) / 8.0).astype(np.float32)
    for tau, T in [(0.5, 64), (1.25, 6), (3.0, 16), (10.0, 3)]:
        oo, pp, ii = oracle.prune_tree(offs, parent, logp, tau, T)
        for b, par in enumerate(parents):
            n = len(par)
            q = np.array([sum(float(logp[offs[b] + a]) for a in synth.root_path(par, i)) for i in range(n)])
            window = sorted([i for i in range(n) if q[i] >= q.max() - tau], key=lambda i: (-q[i], i))[:T]
            got = ii[oo[b]:oo[b + 1]].tolist()
            assert got == sorted(window)
            newpar = pp[oo[b]:oo[b + 1]]
            for r, i in enumerate(got):                # ancestor-closed and re-indexed consistently
                assert (par[i] < 0 and newpar[r] == -1) or got[newpar[r]] == par[i]


def test_stochastic_accept_hand_cases_closed_form_and_level_formulation():
    """The rejection-sampling-style rule of Section 2.1 as a walk over per-node tests."""
    acc = lambda par, pt, pd, u, md=8: [x.tolist() for x in oracle.stochastic_accept(
        np.array([0, len(par)], np.int32), np.asarray(par, np.int32), np.asarray(pt, np.float32),
        np.asarray(pd, np.float32), np.asarray(u, np.float32), md)]
    # chain of 4, ratios p/q = 0.5, 2, 0.25, 1: accepted while u < min(1, p/q)
    par, pt, pd = [-1, 0, 1, 2], [0.25, 0.5, 0.125, 0.5], [0.5, 0.25, 0.5, 0.5]
    assert acc(par, pt, pd, [0.49, 0.99, 0.24, 0.99]) == [[[0, 1, 2, 3, -1, -1, -1, -1]], [4]]
    assert acc(par, pt, pd, [0.49, 0.99, 0.25, 0.0])[1] == [2]          # u == ratio is a rejection (strict <)
    assert acc(par, pt, pd, [0.5, 0.0, 0.0, 0.0])[1] == [0]             # the first test already fails
    assert acc(par, [0, 0, 0, 0], pd, [0, 0, 0, 0])[1] == [0]           # target probability 0 never passes
    # tree: 0 -> {1, 2}, 2 -> {3}; the first passing child in index order is taken, later siblings are not looked at
    par, one = [-1, 0, 0, 2], [1.0] * 4
    assert acc(par, [1, 0.1, 1, 1], one, [0.5, 0.5, 0.5, 0.5]) == [[[0, 2, 3, -1, -1, -1, -1, -1]], [3]]
    assert acc(par, [1, 0.9, 1, 1], one, [0.5, 0.5, 0.5, 0.5]) == [[[0, 1, -1, -1, -1, -1, -1, -1]], [2]]
    assert acc(par, [1, 0.1, 0.1, 1], one, [0.5, 0.5, 0.5, 0.0])[1] == [1]   # node 3 passes but is never reached
    with pytest.raises(ValueError):
        acc([-1, 0, 1], [1, 1, 1], [1, 1, 1], [0, 0, 0], md=2)
    # the acceptance probability of one node is min(1, p/q): sweep u over a grid
    for ptv, pdv in [(0.3, 0.6), (0.6, 0.3), (0.125, 1.0), (0.5, 0.5)]:
        grid = (np.arange(4096) / 4096.0).astype(np.float32)
        n_acc = sum(acc([-1], [ptv], [pdv], [uu])[1][0] for uu in grid[::16])
        assert abs(n_acc / 256.0 - min(1.0, ptv / pdv)) <= 1.0 / 256
    # with it the one-step output distribution equals the target's (speculative sampling's defining property):
    # P(out = x) = q(x) a(x) + (1 - sum_y q(y) a(y)) r(x), a = min(1, p/q), r = normalised max(0, p - q)
    p3, q3 = np.array([0.5, 0.3, 0.2]), np.array([0.2, 0.3, 0.5])
    a3 = np.minimum(1.0, p3 / q3)
    r3 = np.maximum(0.0, p3 - q3)
    np.testing.assert_allclose(q3 * a3 + (1 - (q3 * a3).sum()) * r3 / r3.sum(), p3, atol=1e-15)
    # closed form on chains: p = a q at every node -> P(len >= k) = a^k, so E[len] = a (1 - a^n) / (1 - a)
    rng = np.random.default_rng(77)
    B, n, a = 20000, 6, 0.7
    offs = (np.arange(B + 1) * n).astype(np.int32)
    parent = np.tile(np.arange(-1, n - 1, dtype=np.int32), B)
    pd_ = rng.uniform(0.05, 1.0, B * n).astype(np.float32)
    pt_ = (np.float32(a) * pd_).astype(np.float32)
    _, ln = oracle.stochastic_accept(offs, parent, pt_, pd_, rng.random(B * n, dtype=np.float32), 8)
    mean = a * (1 - a ** n) / (1 - a)
    assert abs(ln.mean() - mean) < 4 * 1.6 / np.sqrt(B)                     # std of the length is below 1.6
    assert abs((ln == n).mean() - a ** n) < 4 * np.sqrt(a ** n * (1 - a ** n) / B)
    # an independent formulation: a node is on the path iff it and all its ancestors pass and have no passing
    # sibling of lower index; resolved for all nodes at once from the parent array
    parents = [synth.random_tree_parent(int(rng.integers(1, 48)), 8, 4, rng) for _ in range(64)]
    offs = np.concatenate([[0], np.cumsum([len(pp) for pp in parents])]).astype(np.int32)
    parent = np.concatenate(parents).astype(np.int32)
    T = int(offs[-1])
    pd_ = rng.uniform(0.05, 1.0, T).astype(np.float32)
    pt_ = rng.uniform(0.0, 1.0, T).astype(np.float32)
    u_ = rng.random(T, dtype=np.float32)
    pi, pl = oracle.stochastic_accept(offs, parent, pt_, pd_, u_, 8)
    passes = (u_ * pd_) < pt_
    for b, par in enumerate(parents):
        ps = passes[offs[b]:offs[b + 1]]
        first = {}                                       # parent -> lowest passing child
        for t in range(len(par)):
            if ps[t]:
                first.setdefault(int(par[t]), t)
        on = [t for t in range(len(par))
              if all(first.get(int(par[x])) == x for x in synth.root_path(par, t))]
        on.sort(key=lambda t: len(synth.root_path(par, t)))
        assert pi[b, :pl[b]].tolist() == on and pl[b] == len(on)


def test_chain_decomposition_paper_example_and_properties():
    """Section 4.3: heavy-light chains.  The chains printed for the paper's example; on random trees the
    chains partition the nodes, each is a path of parent links, a chain hangs off a node of another chain (or
    the committed state), and a root path changes chain at most floor(log2 n) times (the property that
    makes the policy "heavy-light")."""
    parent, chains = {}, []
    for line in open(os.path.join(GOLDEN, "hld_example.txt")):
        tok = line.split()
        if not tok or tok[0].startswith("#"):
            continue
        if tok[0] == "parent":
            parent = {int(a.split(":")[0]): int(a.split(":")[1]) for a in tok[1:]}
        elif tok[0] == "chain":
            chains.append([int(x) for x in tok[1:]])
    n = len(parent)
    par = np.array([parent[i + 1] - 1 for i in range(n)], np.int32)          # 1-based, 0 = committed state -> local, -1
    head, cnt = oracle.chain_decompose(np.array([0, n], np.int32), par)
    got = {}
    for t in range(n):
        got.setdefault(int(head[t]) + 1, []).append(t + 1)
    assert sorted(got.values()) == sorted(chains) and cnt.tolist() == [len(chains)]
    # hand case with a tie and a forest: 0 -> {1, 2} (equal subtrees: the lower index is heavy), second root 3
    head, cnt = oracle.chain_decompose(np.array([0, 5], np.int32), np.array([-1, 0, 0, -1, 3], np.int32))
    assert head.tolist() == [0, 0, 2, 3, 3] and cnt.tolist() == [3]
    rng = np.random.default_rng(91)
    parents = [synth.random_tree_parent(int(rng.integers(1, 65)), 8, 4, rng) for _ in range(40)]
    parents += [synth.chain_parent(8), np.zeros(0, np.int32), synth.proposal_tree_parent(2, 14, 30, rng, 16)]
    offs = np.concatenate([[0], np.cumsum([len(pp) for pp in parents])]).astype(np.int32)
    head, cnt = oracle.chain_decompose(offs, np.concatenate(parents).astype(np.int32))
    for b, par in enumerate(parents):
        n = len(par)
        h = head[offs[b]:offs[b + 1]]
        members = {}
        for t in range(n):
            members.setdefault(int(h[t]), []).append(t)
        assert cnt[b] == len(members) and all(k == v[0] for k, v in members.items())
        size = [len([t for t in range(n) if i in synth.root_path(par, t)]) for i in range(n)]      # brute force
        for k, v in members.items():
            for a_, b_ in zip(v, v[1:]):
                assert par[b_] == a_                                                      # a path of parent links
                sib = [t for t in range(n) if par[t] == a_]
                assert size[b_] == max(size[t] for t in sib)                               # along the heaviest child
                assert b_ == min(t for t in sib if size[t] == size[b_])                    # lowest index on ties
            assert par[k] < 0 or h[par[k]] != k                                           # the head hangs off another chain
        for t in range(n):
            path = synth.root_path(par, t)
            changes = sum(1 for a_, b_ in zip(path, path[1:]) if h[a_] != h[b_])
            assert changes <= int(np.floor(np.log2(n)))


def test_rule_without_erase_is_gated_linear_attention():
    """Rule 1 (GLA-style records, Section 5.1 remark): S' = alpha S + beta v k^T.  Closed form along a path:
    S_t = gamma_t S0 + sum_{i on path} (gamma_t / gamma_i) beta_i v_i k_i^T, evaluated directly with numpy for
    every node of a tree; commit over a path likewise.  The default rule is restored afterwards."""
    rng = np.random.default_rng(71)
    par = synth.random_tree_parent(12, 5, 3, rng)
    prob = synth.make_problem(71, 2, 2, 16, 8, [par])
    try:
        oracle.set_rule(oracle.RULE_GATED_NO_ERASE)
        o = run_verify(prob)
        path = synth.root_path(par, 11)
        idx = np.full((1, 8), -1, np.int32); idx[0, :len(path)] = path
        Sc = oracle.commit(prob.S0, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets, idx,
                           np.array([len(path)], np.int32))
    finally:
        oracle.set_rule(oracle.RULE_GATED_DELTA)
    for l in range(2):
        for h in range(2):
            S0, q, k, v, al, be, _ = unit_arrays(prob, l=l, b=0, h=h)
            def state(t):
                pth = synth.root_path(par, t)
                gam = np.cumprod([al[i] for i in pth])
                S = gam[-1] * S0
                for j, i in enumerate(pth):
                    S = S + (gam[-1] / gam[j]) * be[i] * np.outer(v[i], k[i])
                return S
            for t in range(12):
                assert np.allclose(state(t) @ q[t], o[l, t, h], rtol=1e-12, atol=1e-14)
            assert np.allclose(state(11), Sc[l, 0, h], rtol=1e-12, atol=1e-14)
    assert not np.allclose(run_verify(prob), o)          # and it is a different rule from the default one


def test_paper_byte_counts():
    vals = {}
    for r in open(os.path.join(GOLDEN, "paper_sizes.txt")):
        if r.strip() and not r.startswith("#"):
            key, val = r.split()[:2]
            vals[key] = float(val)
    MiB, KiB = 1024 * 1024, 1024
    state = lambda h, dk, dv: 4 * h * dk * dv
    assert state(8, 256, 256) == vals["state_MiB_per_layer"] * MiB
    assert state(32, 128, 128) == vals["state_MiB_per_layer"] * MiB
    assert 2 * state(8, 256, 256) == vals["round_trip_MiB_per_token"] * MiB
    assert 8 * state(8, 256, 256) == vals["snapshots_MiB_L8"] * MiB
    record = lambda h, dk, dv: 4 * h * (dk + dv + 2)          # fp32 {k, v, alpha, beta} per head
    assert 8 * record(8, 256, 256) == vals["factor_buffer_KiB_L8"] * KiB
    assert abs(state(8, 256, 256) / record(8, 256, 256) - vals["snapshot_over_factor_ratio"]) < 1.0
