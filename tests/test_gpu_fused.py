"""GPU parity of the fused commit-and-verify entry point (delayed state update, Section 5.2):
speca_commit_verify_tree must equal the oracle's commit followed by the oracle's verify, on
the state it writes back and on the outputs of the new draft."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth
from gpu_util import DevProblem, TOL, TOL_FP32, rel_err, tol_for

pytestmark = pytest.mark.gpu


def cpu(t):
    return t.detach().cpu().numpy()


def random_paths(rng, prob, zero_frac=0.25):
    """Prescribe a random root path (or nothing, with probability zero_frac) per sequence."""
    paths = []
    for b in range(prob.B):
        lo, hi = int(prob.node_offsets[b]), int(prob.node_offsets[b + 1])
        if hi == lo or rng.random() < zero_frac:
            paths.append([])
        else:
            paths.append(synth.root_path(prob.parent[lo:hi], int(rng.integers(0, hi - lo))))
    synth._set_paths(prob, paths)


def prev_dict(dp, with_u=True, with_parent=True):
    return dict(k=dp.k, v=dp.v, alpha=dp.alpha, beta=dp.beta, u=dp.u if with_u else None,
                node_offsets=dp.node_offsets, total_nodes=dp.T, parent=dp.parent if with_parent else None)


def fused_call(d_new, S, prev, path_idx, path_len):
    speca.commit_verify_tree(d_new.dims, S, prev, path_idx, path_len, d_new.q, d_new.k, d_new.v, d_new.alpha,
                             d_new.beta, d_new.node_offsets, d_new.T, d_new.parent, d_new.depth, d_new.o, d_new.u,
                             d_new.ws, d_new.status)


def oracle_commit_then_verify(S, p_prev, p_new):
    S1 = oracle.commit(S, p_prev.k, p_prev.v, p_prev.alpha, p_prev.beta, p_prev.node_offsets, p_prev.path_idx,
                       p_prev.path_len)
    o = oracle.verify_tree(S1, p_new.q, p_new.k, p_new.v, p_new.alpha, p_new.beta, p_new.node_offsets, p_new.parent)
    return S1, o


def run_pair(seed, L, H, d_k, d_v, parents_prev, parents_new, route, state_std=0.02, with_u=True, max_nodes=64):
    """Verify draft 1 (to get its u), then commit its prescribed paths and verify draft 2 in one call."""
    rng = np.random.default_rng(seed)
    p1 = synth.make_problem(seed, L, H, d_k, d_v, parents_prev, state_std=state_std, name="prev")
    p2 = synth.make_problem(seed + 1, L, H, d_k, d_v, parents_new, state_std=state_std, name="new")
    random_paths(rng, p1)
    d1 = DevProblem(p1, route=route, want_u=True, max_nodes=max_nodes)
    d1.verify_tree()
    assert d1.status_value() == 0
    d2 = DevProblem(p2, route=route, want_u=True, max_nodes=max_nodes)
    S = d1.S.clone()
    fused_call(d2, S, prev_dict(d1, with_u), d1.path_idx, d1.path_len)
    assert d2.status_value() == 0
    S_ref, o_ref = oracle_commit_then_verify(p1.S0, p1, p2)
    return p1, p2, d1, d2, S, S_ref, o_ref


CASES = [
    # name, L, H, d_v, previous draft, new draft
    ("chains", 2, 4, 128, lambda r: [synth.chain_parent(8)] * 3, lambda r: [synth.chain_parent(8)] * 3),
    ("trees-256", 2, 4, 256, lambda r: synth.ragged_tree_batch(r, 6, 8, 64, 8), lambda r: synth.ragged_tree_batch(r, 6, 8, 64, 8)),
    ("trees-128", 3, 16, 128, lambda r: synth.ragged_tree_batch(r, 4, 32, 32, 6), lambda r: synth.ragged_tree_batch(r, 4, 32, 32, 6)),
    ("ragged-mix", 2, 4, 256,
     lambda r: [synth.random_tree_parent(64, 8, 4, r), synth.chain_parent(8), synth.chain_parent(3), np.zeros(0, np.int32),
                synth.chain_parent(1)],
     lambda r: [synth.random_tree_parent(40, 8, 4, r), np.zeros(0, np.int32), synth.chain_parent(8), synth.chain_parent(2),
                synth.random_tree_parent(17, 5, 3, r)]),
]


@pytest.mark.parametrize("route", [speca.ROUTE_TF32, speca.ROUTE_AUTO], ids=["one-pass-tf32", "auto"])
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_fused_equals_commit_then_verify(case, route):
    """ROUTE_TF32: the one-pass kernel (state read once as TF32).  AUTO: the commit kernel followed by the
    fp32-grade verification, held to the fp32 bar."""
    name, L, H, d_v, mk_prev, mk_new = case
    rng = np.random.default_rng(11)
    p1, p2, d1, d2, S, S_ref, o_ref = run_pair(21, L, H, 128, d_v, mk_prev(rng), mk_new(rng), route)
    assert rel_err(cpu(S), S_ref) <= tol_for(route), name
    assert rel_err(cpu(d2.o), o_ref) <= tol_for(route), name
    # sequences without an accepted path keep their state bit for bit
    for b in np.flatnonzero(p1.path_len == 0):
        assert torch.equal(S[:, b], d1.S[:, b])
    # and the state that IS advanced agrees with the stand-alone commit kernel to fp32 accuracy
    d1.commit()
    assert d1.status_value() == 0
    assert rel_err(cpu(S), cpu(d1.S)) <= 1e-4


@pytest.mark.parametrize("route,with_u,tol", [(speca.ROUTE_SERIAL, True, TOL_FP32), (speca.ROUTE_TF32, False, TOL),
                                              (speca.ROUTE_FACTORIZED, True, TOL_FP32), (speca.ROUTE_AUTO, True, TOL_FP32)])
def test_fused_fallbacks_give_the_same_results(route, with_u, tol):
    """Serial route, or no u from the previous verification: the two kernels run back to back."""
    rng = np.random.default_rng(5)
    parents = synth.ragged_tree_batch(rng, 5, 4, 40, 8)
    p1, p2, d1, d2, S, S_ref, o_ref = run_pair(31, 2, 2, 128, 128, parents, synth.ragged_tree_batch(rng, 5, 4, 40, 8),
                                               route, with_u=with_u)
    assert rel_err(cpu(d2.o), o_ref) <= tol
    assert rel_err(cpu(S), S_ref) <= (TOL_FP32 if (route == speca.ROUTE_SERIAL or not with_u) else TOL)


def test_fused_shapes_outside_the_tensor_core_route():
    """d_k = 64: the entry point still works (commit kernel, then the state-resident verify)."""
    rng = np.random.default_rng(6)
    p1, p2, d1, d2, S, S_ref, o_ref = run_pair(41, 1, 4, 64, 64, [synth.chain_parent(4)] * 2,
                                               [synth.random_tree_parent(9, 4, 3, rng)] * 2, speca.ROUTE_AUTO, max_nodes=16)
    assert rel_err(cpu(d2.o), o_ref) <= TOL_FP32
    assert rel_err(cpu(S), S_ref) <= TOL_FP32


@pytest.mark.parametrize("d_v", [128, 256])
def test_fused_key_width_256(d_v):
    """The paper's target shape on the single-pass kernel (up to 32 nodes per sequence)."""
    rng = np.random.default_rng(13 + d_v)
    prev = synth.ragged_tree_batch(rng, 5, 4, 32, 8) + [synth.chain_parent(8), np.zeros(0, np.int32)]
    new = synth.ragged_tree_batch(rng, 5, 4, 32, 8) + [np.zeros(0, np.int32), synth.chain_parent(8)]
    p1, p2, d1, d2, S, S_ref, o_ref = run_pair(45, 2, 8, 256, d_v, prev, new, speca.ROUTE_TF32, max_nodes=32)
    assert rel_err(cpu(d2.o), o_ref) <= TOL
    assert rel_err(cpu(S), S_ref) <= TOL
    d1.commit()
    assert rel_err(cpu(S), cpu(d1.S)) <= 1e-4
    for b in np.flatnonzero(p1.path_len == 0):
        assert torch.equal(S[:, b], d1.S[:, b])


def test_nothing_pending_and_nothing_to_verify():
    rng = np.random.default_rng(8)
    prob = synth.make_problem(51, 2, 4, 128, 256, synth.ragged_tree_batch(rng, 3, 8, 30, 8))
    random_paths(rng, prob, zero_frac=0.0)
    # first round: no previous draft -> plain verification, S is not written
    dp = DevProblem(prob, route=speca.ROUTE_TF32, want_u=True, max_nodes=64)
    S = dp.S.clone()
    fused_call(dp, S, None, dp.path_idx, dp.path_len)
    assert dp.status_value() == 0 and torch.equal(S, dp.S)
    o_ref = oracle.verify_tree(prob.S0, prob.q, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets, prob.parent)
    assert rel_err(cpu(dp.o), o_ref) <= TOL
    # last round: nothing left to verify -> plain commit of the pending paths
    empty = synth.make_problem(52, 2, 4, 128, 256, [np.zeros(0, np.int32)] * 3)
    de = DevProblem(empty, route=speca.ROUTE_TF32, want_u=True, max_nodes=64)
    fused_call(de, S, prev_dict(dp), dp.path_idx, dp.path_len)
    assert de.status_value() == 0
    S_ref = oracle.commit(prob.S0, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets, prob.path_idx, prob.path_len)
    assert rel_err(cpu(S), S_ref) <= TOL_FP32


def test_bad_pending_path_skips_only_that_commit():
    """A pending path that is not a parent chain: status bit, that sequence's state stays as it was
    and its new draft is verified from it; the other sequences are committed and verified."""
    rng = np.random.default_rng(9)
    parents = [synth.chain_parent(6), synth.chain_parent(6), synth.random_tree_parent(20, 6, 3, rng)]
    p1 = synth.make_problem(61, 1, 4, 128, 256, parents)
    p2 = synth.make_problem(62, 1, 4, 128, 256, [synth.chain_parent(5)] * 3)
    synth._set_paths(p1, [[0, 1, 2], [0, 2, 3], synth.root_path(parents[2], 19)])      # sequence 1: 2 is not a child of 0
    d1 = DevProblem(p1, route=speca.ROUTE_TF32, want_u=True, max_nodes=64)
    d1.verify_tree()
    d2 = DevProblem(p2, route=speca.ROUTE_TF32, want_u=True, max_nodes=64)
    S = d1.S.clone()
    fused_call(d2, S, prev_dict(d1), d1.path_idx, d1.path_len)
    assert d2.status_value() == speca.STATUS_BAD_PATH
    good = p1.path_len.copy(); good[1] = 0
    S_ref = oracle.commit(p1.S0, p1.k, p1.v, p1.alpha, p1.beta, p1.node_offsets, p1.path_idx, good)
    o_ref = oracle.verify_tree(S_ref, p2.q, p2.k, p2.v, p2.alpha, p2.beta, p2.node_offsets, p2.parent)
    assert torch.equal(S[:, 1], d1.S[:, 1])
    assert rel_err(cpu(S), S_ref) <= TOL
    assert rel_err(cpu(d2.o), o_ref) <= TOL
    # without the parent array nothing can be checked: valid root paths are applied as given
    synth._set_paths(p1, [[0, 1, 2], [0, 1, 2, 3], synth.root_path(parents[2], 19)])
    d1.path_idx.copy_(torch.from_numpy(p1.path_idx).cuda())
    d1.path_len.copy_(torch.from_numpy(p1.path_len).cuda())
    d2.status.zero_()
    S = d1.S.clone()
    fused_call(d2, S, prev_dict(d1, with_parent=False), d1.path_idx, d1.path_len)
    assert d2.status_value() == 0
    S_ref = oracle.commit(p1.S0, p1.k, p1.v, p1.alpha, p1.beta, p1.node_offsets, p1.path_idx, p1.path_len)
    assert rel_err(cpu(S), S_ref) <= TOL


def test_rejected_new_tree_still_gets_its_commit():
    rng = np.random.default_rng(10)
    p1 = synth.make_problem(71, 1, 4, 128, 128, [synth.chain_parent(4)] * 2)
    p2 = synth.make_problem(72, 1, 4, 128, 128, [synth.chain_parent(4)] * 2)
    synth._set_paths(p1, [[0, 1], [0, 1, 2]])
    p2.parent[5] = 3                      # sequence 1, local node 1: parent 3 >= 1 is not topological
    d1 = DevProblem(p1, route=speca.ROUTE_TF32, want_u=True, max_nodes=64)
    d1.verify_tree()
    d2 = DevProblem(p2, route=speca.ROUTE_TF32, want_u=True, max_nodes=64)
    S = d1.S.clone()
    speca.commit_verify_tree(d2.dims, S, prev_dict(d1), d1.path_idx, d1.path_len, d2.q, d2.k, d2.v, d2.alpha, d2.beta,
                             d2.node_offsets, d2.T, d2.parent, None, d2.o, d2.u, d2.ws, d2.status)
    assert d2.status_value() == speca.STATUS_BAD_PARENT
    S_ref = oracle.commit(p1.S0, p1.k, p1.v, p1.alpha, p1.beta, p1.node_offsets, p1.path_idx, p1.path_len)
    assert rel_err(cpu(S), S_ref) <= TOL
    assert torch.isnan(d2.o[:, 4:]).all()                     # the rejected sequence's outputs are left untouched
    p2.parent[5] = 0
    o_ref = oracle.verify_tree(S_ref, p2.q, p2.k, p2.v, p2.alpha, p2.beta, p2.node_offsets, p2.parent)
    assert rel_err(cpu(d2.o[:, :4]), o_ref[:, :4]) <= TOL


def test_fused_rounds_carry_the_state():
    """Six rounds of fused verify -> accept with the commit delayed into the next round, then a flush."""
    rng = np.random.default_rng(12)
    L, H, B = 2, 4, 6
    probs = []
    for r in range(6):
        parents = synth.mixed_chain_tree_batch(rng, B, 8, 48, 8) if r % 2 == 0 else synth.ragged_tree_batch(rng, B, 4, 64, 8)
        probs.append(synth.make_problem(100 + r, L, H, 128, 256, parents))
    devs = [DevProblem(p, route=speca.ROUTE_TF32, want_u=True, max_nodes=64) for p in probs]
    S = devs[0].S.clone()
    S_ref = probs[0].S0.astype(np.float64)
    prev = None
    worst_o = 0.0
    for r, (p, d) in enumerate(zip(probs, devs)):
        pd = devs[r - 1] if r else d
        fused_call(d, S, prev, pd.path_idx, pd.path_len)
        d.accept()
        assert d.status_value() == 0
        if r:
            pp = probs[r - 1]
            S_ref = oracle.commit(S_ref, pp.k, pp.v, pp.alpha, pp.beta, pp.node_offsets, cpu(pd.path_idx), cpu(pd.path_len))
        o_ref = oracle.verify_tree(S_ref, p.q, p.k, p.v, p.alpha, p.beta, p.node_offsets, p.parent)
        pi, pl, _ = oracle.greedy_accept(p.node_offsets, p.parent, p.draft_tok, p.target_tok, p.root_target_tok, 8)
        assert np.array_equal(cpu(d.path_idx), pi) and np.array_equal(cpu(d.path_len), pl)
        worst_o = max(worst_o, rel_err(cpu(d.o), o_ref))
        assert rel_err(cpu(S), S_ref) <= TOL
        prev = prev_dict(d)
    assert worst_o <= TOL, worst_o
    # flush the last pending commit with the stand-alone kernel
    last, pl = devs[-1], probs[-1]
    speca.commit(last.dims, S, last.k, last.v, last.alpha, last.beta, last.node_offsets, last.T, last.parent,
                 last.path_idx, last.path_len, last.status)
    S_ref = oracle.commit(S_ref, pl.k, pl.v, pl.alpha, pl.beta, pl.node_offsets, cpu(last.path_idx), cpu(last.path_len))
    assert rel_err(cpu(S), S_ref) <= TOL


def test_more_sequences_than_the_walk_table_holds():
    """Batches beyond the kernel's shared-memory walk table (128 sequences) take the global-memory
    path for the per-sequence data: plain verification and the fused call on 150 sequences."""
    rng = np.random.default_rng(17)
    B = 150
    prev = [synth.random_tree_parent(int(rng.integers(1, 13)), 4, 3, rng) for _ in range(B)]
    new = [synth.random_tree_parent(int(rng.integers(1, 13)), 4, 3, rng) for _ in range(B)]
    new[140] = np.zeros(0, np.int32)
    p1, p2, d1, d2, S, S_ref, o_ref = run_pair(47, 1, 2, 128, 128, prev, new, speca.ROUTE_TF32, max_nodes=16)
    o1_ref = oracle.verify_tree(p1.S0, p1.q, p1.k, p1.v, p1.alpha, p1.beta, p1.node_offsets, p1.parent)
    assert rel_err(cpu(d1.o), o1_ref) <= TOL
    assert rel_err(cpu(d2.o), o_ref) <= TOL
    assert rel_err(cpu(S), S_ref) <= TOL


def _banded(t, pad=256, fill=7.5):
    """A copy of tensor t placed in the middle of a larger buffer filled with a sentinel."""
    flat = torch.full((t.numel() + 2 * pad,), fill, dtype=t.dtype, device=t.device)
    flat[pad:pad + t.numel()] = t.flatten()
    return flat, flat[pad:pad + t.numel()].view_as(t)


def test_tensor_core_kernels_write_nothing_outside_their_tensors():
    """Guard bands around everything the tensor-core kernels write (o, u, and S for the fused call, which goes
    back through TMA stores): the sentinel values on both sides must survive."""
    rng = np.random.default_rng(19)
    p1 = synth.make_problem(191, 2, 3, 128, 256, synth.ragged_tree_batch(rng, 3, 5, 40, 8))
    p2 = synth.make_problem(192, 2, 3, 128, 256, synth.ragged_tree_batch(rng, 3, 5, 40, 8))
    random_paths(rng, p1, zero_frac=0.0)
    d1 = DevProblem(p1, route=speca.ROUTE_TF32, want_u=True, max_nodes=64)
    bo, d1.o = _banded(d1.o)
    bu, d1.u = _banded(d1.u)
    d1.verify_tree()
    d2 = DevProblem(p2, route=speca.ROUTE_TF32, want_u=True, max_nodes=64)
    bo2, d2.o = _banded(d2.o)
    bu2, d2.u = _banded(d2.u)
    bS, S = _banded(d1.S)
    fused_call(d2, S, prev_dict(d1), d1.path_idx, d1.path_len)
    assert d1.status_value() == 0 and d2.status_value() == 0
    for band in (bo, bu, bo2, bu2, bS):
        assert torch.all(band[:256] == 7.5) and torch.all(band[-256:] == 7.5)
    S_ref, o_ref = oracle_commit_then_verify(p1.S0, p1, p2)
    assert rel_err(cpu(S), S_ref) <= TOL and rel_err(cpu(d2.o), o_ref) <= TOL
