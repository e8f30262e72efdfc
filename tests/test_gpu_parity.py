"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by
element, on the same seeded inputs."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth
from gpu_util import DevProblem, TOL, TOL_FP32, oracle_commit, oracle_verify, rel_err, tol_for

pytestmark = pytest.mark.gpu

# the serial walk, the tensor-core routes with split operands (factorised, effective-query) and the single-pass
# TF32 route; each is held to its own bar (gpu_util.tol_for)
ROUTES = [speca.ROUTE_SERIAL, speca.ROUTE_FACTORIZED, speca.ROUTE_EFFECTIVE, speca.ROUTE_TF32]


def cpu(t):
    return t.detach().cpu().numpy()


def check_verify(prob, route, chain=False, tol=None, want_u=False, max_nodes=None):
    tol = tol_for(route) if tol is None else tol
    dp = DevProblem(prob, route=route, want_u=want_u, max_nodes=max_nodes)
    S_before = dp.S.clone()
    o = dp.verify_chain() if chain else dp.verify_tree()
    assert dp.status_value() == 0
    assert torch.equal(dp.S, S_before), "verify must leave the committed state bitwise unchanged"
    ref = oracle_verify(prob)
    e = rel_err(cpu(o), ref)
    assert e <= tol and e <= TOL, f"{prob.name}: verify error {e:.3e}"
    return dp, ref


# ---------------------------------------------------------------------------
# configuration 1: tiny chain, also against decode steps
# ---------------------------------------------------------------------------
def test_unsupported_shapes_fall_back_or_are_refused():
    """d_k = 64 is outside the factorised route: AUTO takes the serial route, an explicit request is refused."""
    prob = synth.config(1)
    dp, _ = check_verify(prob, speca.ROUTE_AUTO, chain=True, tol=TOL_FP32)
    dp = DevProblem(prob, route=speca.ROUTE_FACTORIZED)
    with pytest.raises(speca.SpecaError, match="unsupported"):
        dp.verify_tree()


@pytest.mark.parametrize("route", [speca.ROUTE_SERIAL])
def test_cfg1_chain_verify_commit_and_decode(route):
    prob = synth.config(1)
    dp, ref = check_verify(prob, route, chain=True)
    o_chain = dp.o.clone()
    dp.o.fill_(float("nan"))
    dp.verify_tree()
    assert rel_err(cpu(dp.o), ref) <= tol_for(route)             # single-path tree == chain
    # commit the first two tokens
    dp.commit()
    assert dp.status_value() == 0
    S_ref = oracle_commit(prob, prob.path_idx, prob.path_len)
    assert rel_err(cpu(dp.S), S_ref) <= TOL_FP32
    # the same tokens by single-token decode steps
    d1 = speca.Dims(prob.L, 1, prob.H, prob.d_k, prob.d_v)
    S = torch.from_numpy(prob.S0).cuda()
    So = prob.S0.astype(np.float64)
    for t in range(prob.T):
        o = torch.empty(prob.L, 1, prob.H, prob.d_v, device="cuda")
        speca.decode_step(d1, S, dp.q[:, t:t + 1].contiguous(), dp.k[:, t:t + 1].contiguous(),
                          dp.v[:, t:t + 1].contiguous(), dp.alpha[:, t:t + 1].contiguous(),
                          dp.beta[:, t:t + 1].contiguous(), o)
        So, oo = oracle.decode_step(So, prob.q[:, t:t + 1], prob.k[:, t:t + 1], prob.v[:, t:t + 1],
                                    prob.alpha[:, t:t + 1], prob.beta[:, t:t + 1])
        assert rel_err(cpu(o), oo) <= TOL_FP32
        assert rel_err(cpu(S), So) <= TOL_FP32
        assert rel_err(cpu(o[:, 0]), cpu(o_chain[:, t])) <= TOL_FP32
        if t == 1:
            assert rel_err(cpu(S), cpu(dp.S)) <= TOL_FP32         # commit of 2 == 2 decode steps


# ---------------------------------------------------------------------------
# configuration 2: 24 layers x 16 heads, chain of 8, accepted length 0..8
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("route", ROUTES)
@pytest.mark.parametrize("accepted", [None, 0, 8])
def test_cfg2_chain(route, accepted):
    prob = synth.config(2)
    if accepted is not None:
        synth._set_paths(prob, [list(range(accepted))])
    dp, _ = check_verify(prob, route, chain=True)
    S_before = dp.S.clone()
    dp.commit()
    assert dp.status_value() == 0
    if int(prob.path_len[0]) == 0:
        assert torch.equal(dp.S, S_before)
    S_ref = oracle_commit(prob, prob.path_idx, prob.path_len)
    assert rel_err(cpu(dp.S), S_ref) <= TOL_FP32


def test_cfg2_chain_equals_eight_decode_steps():
    prob = synth.config(2)
    dp = DevProblem(prob, route=speca.ROUTE_SERIAL)
    o_chain = cpu(dp.verify_chain()).copy()
    d1 = speca.Dims(prob.L, 1, prob.H, prob.d_k, prob.d_v)
    S = dp.S.clone()
    for t in range(8):
        o = torch.empty(prob.L, 1, prob.H, prob.d_v, device="cuda")
        speca.decode_step(d1, S, dp.q[:, t:t + 1].contiguous(), dp.k[:, t:t + 1].contiguous(),
                          dp.v[:, t:t + 1].contiguous(), dp.alpha[:, t:t + 1].contiguous(),
                          dp.beta[:, t:t + 1].contiguous(), o)
        assert rel_err(cpu(o[:, 0]), o_chain[:, t]) <= TOL_FP32
    synth._set_paths(prob, [list(range(8))])
    dp2 = DevProblem(prob, route=speca.ROUTE_SERIAL)
    dp2.commit()
    assert rel_err(cpu(dp2.S), cpu(S)) <= TOL_FP32


# ---------------------------------------------------------------------------
# configuration 3: 32-node tree, random root-to-leaf path committed
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("route", ROUTES)
def test_cfg3_tree(route):
    prob = synth.config(3)
    dp, _ = check_verify(prob, route, want_u=True)
    dp.commit()
    assert dp.status_value() == 0
    S_ref = oracle_commit(prob, prob.path_idx, prob.path_len)
    assert rel_err(cpu(dp.S), S_ref) <= TOL_FP32
    # u is the WY-style factor: S_t = gamma_t S0 + sum (gamma_t/gamma_i) u_i k_i^T rebuilds the committed state
    tol = tol_for(route)
    l, h = 3, 5
    path = prob.path_idx[0, :prob.path_len[0]]
    S = prob.S0[l, 0, h].astype(np.float64)
    u = cpu(dp.u)[l, :, h].astype(np.float64)
    kf = synth.bf16_bits_to_f32(prob.k[l, :, h]).astype(np.float64)
    for t in path:
        S = prob.alpha[l, t, h].astype(np.float64) * S + np.outer(u[t], kf[t])
    assert rel_err(S, S_ref[l, 0, h]) <= tol


# ---------------------------------------------------------------------------
# configuration 4 (reduced layers, full batch of ragged trees): verify -> accept -> commit
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("route", ROUTES)
def test_cfg4_reduced_full_compare(route):
    prob = synth.config(4, L=2)
    dp, _ = check_verify(prob, route)
    dp.accept()
    pi, pl, nt = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                      prob.root_target_tok, prob.max_depth)
    assert dp.status_value() == 0
    assert np.array_equal(cpu(dp.path_idx), pi) and np.array_equal(cpu(dp.path_len), pl)
    assert np.array_equal(cpu(dp.next_tok), nt)
    assert pl.max() >= 2
    dp.commit()
    assert dp.status_value() == 0
    assert rel_err(cpu(dp.S), oracle_commit(prob, pi, pl)) <= TOL_FP32


# ---------------------------------------------------------------------------
# shapes: every supported d_k, several d_v, tiles with ragged tails
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("d_k,d_v", [(64, 32), (64, 96), (128, 160), (256, 64), (256, 256), (128, 1024)])
def test_shapes(d_k, d_v):
    rng = np.random.default_rng(d_k + d_v)
    parents = [synth.random_tree_parent(19, 6, 3, rng), synth.chain_parent(5), synth.random_tree_parent(33, 8, 4, rng)]
    prob = synth.make_problem(d_k * 7 + d_v, 2, 3, d_k, d_v, parents, state_std=0.5, name=f"shape{d_k}x{d_v}")
    prob.scale = 0.125
    dp, _ = check_verify(prob, speca.ROUTE_SERIAL, want_u=True)
    dp.accept()
    pi, pl, nt = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                      prob.root_target_tok, prob.max_depth)
    assert np.array_equal(cpu(dp.path_idx), pi) and np.array_equal(cpu(dp.path_len), pl)
    dp.commit()
    assert rel_err(cpu(dp.S), oracle_commit(prob, pi, pl)) <= TOL_FP32
    # decode step on the same shapes
    L, B, H = prob.L, prob.B, prob.H
    q, k, v, al, be = synth.draw_records(rng, L, B, H, d_k, d_v)
    d1 = speca.Dims(L, B, H, d_k, d_v, scale=0.125)
    from gpu_util import bf16_dev
    S = torch.from_numpy(prob.S0).cuda()
    o = torch.empty(L, B, H, d_v, device="cuda")
    speca.decode_step(d1, S, bf16_dev(q), bf16_dev(k), bf16_dev(v), torch.from_numpy(al).cuda(),
                      torch.from_numpy(be).cuda(), o)
    Sr, orf = oracle.decode_step(prob.S0, q, k, v, al, be, scale=0.125)
    assert rel_err(cpu(S), Sr) <= TOL_FP32 and rel_err(cpu(o), orf) <= TOL_FP32


# ---------------------------------------------------------------------------
# edge cases
# ---------------------------------------------------------------------------
def test_empty_sequences_single_nodes_and_forests():
    rng = np.random.default_rng(77)
    forest = np.array([-1, -1, 0, -1, 1, 1, 2, 3, 3, 6], np.int32)       # three roots
    stars = np.array([-1] * 6, np.int32)                                   # "all-root" proposal
    parents = [np.zeros(0, np.int32), synth.chain_parent(1), forest, np.zeros(0, np.int32), stars,
               synth.random_tree_parent(64, 8, 4, rng)]
    prob = synth.make_problem(78, 2, 2, 128, 64, parents, state_std=0.3)
    dp, _ = check_verify(prob, speca.ROUTE_SERIAL)
    dp.accept()
    pi, pl, nt = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                      prob.root_target_tok, prob.max_depth)
    assert np.array_equal(cpu(dp.path_idx), pi) and np.array_equal(cpu(dp.path_len), pl)
    assert np.array_equal(cpu(dp.next_tok), nt)
    assert pl[0] == 0 and pl[3] == 0
    S_before = dp.S.clone()
    dp.commit()
    assert dp.status_value() == 0
    assert rel_err(cpu(dp.S), oracle_commit(prob, pi, pl)) <= TOL_FP32
    for b in np.flatnonzero(pl == 0):
        assert torch.equal(dp.S[:, int(b)], S_before[:, int(b)])


def test_maximum_depth_and_node_budget():
    rng = np.random.default_rng(5)
    parents = [synth.chain_parent(16), synth.random_tree_parent(200, 16, 4, rng)]
    prob = synth.make_problem(6, 1, 2, 64, 64, parents, max_depth=16, state_std=0.2)
    synth._set_paths(prob, [list(range(16)), synth.root_path(parents[1], 199)])
    dp, _ = check_verify(prob, speca.ROUTE_SERIAL)
    dp.commit()
    assert dp.status_value() == 0
    assert rel_err(cpu(dp.S), oracle_commit(prob, prob.path_idx, prob.path_len)) <= TOL_FP32


def test_device_side_faults_set_status_and_skip_the_sequence():
    rng = np.random.default_rng(9)
    parents = [synth.random_tree_parent(12, 5, 3, rng) for _ in range(4)]
    prob = synth.make_problem(10, 1, 2, 64, 64, parents)
    good = oracle_verify(prob)
    s1, e1 = int(prob.node_offsets[1]), int(prob.node_offsets[2])
    # (a) forward parent pointer in sequence 1
    bad = synth.make_problem(10, 1, 2, 64, 64, parents)
    bad.parent[s1 + 3] = 7
    dp = DevProblem(bad, route=speca.ROUTE_SERIAL)
    dp.verify_tree(with_depth=False)
    assert dp.status_value() & speca.STATUS_BAD_PARENT
    o = cpu(dp.o)
    assert np.all(np.isnan(o[:, s1:e1]))                               # skipped: outputs untouched
    keep = np.r_[0:s1, e1:prob.T]
    assert rel_err(o[:, keep], good[:, keep]) <= TOL_FP32
    dp.status.zero_()
    dp.accept()
    assert dp.status_value() & speca.STATUS_BAD_PARENT and int(dp.path_len[1]) == 0
    # (b) node budget exceeded by one sequence only: that sequence is skipped, the rest is computed
    big = synth.make_problem(12, 1, 2, 64, 64, [parents[0], synth.random_tree_parent(20, 5, 3, rng), parents[2]])
    dp = DevProblem(big, route=speca.ROUTE_SERIAL, max_nodes=16)
    dp.verify_tree()
    assert dp.status_value() & speca.STATUS_TOO_MANY
    o, ref = cpu(dp.o), oracle_verify(big)
    assert np.all(np.isnan(o[:, 12:32]))
    keep = np.r_[0:12, 32:44]
    assert rel_err(o[:, keep], ref[:, keep]) <= TOL_FP32
    dp.o.fill_(float("nan")); dp.status.zero_()
    dp.verify_chain()                                   # the chain entry point applies the same budget
    assert dp.status_value() & speca.STATUS_TOO_MANY and np.all(np.isnan(cpu(dp.o)[:, 12:32]))
    # (c) deeper than max_depth
    deep = synth.make_problem(11, 1, 1, 64, 64, [synth.chain_parent(6)], max_depth=4)
    dp = DevProblem(deep, route=speca.ROUTE_SERIAL)
    dp.verify_tree()
    assert dp.status_value() & speca.STATUS_TOO_DEEP
    # (d) inconsistent depth[] is reported
    dp = DevProblem(prob, route=speca.ROUTE_SERIAL)
    dp.depth[2] += 1
    dp.verify_tree()
    assert dp.status_value() & speca.STATUS_BAD_DEPTH
    # (e) commit: path that is not a parent chain, and over-long path: state untouched
    dp = DevProblem(prob, route=speca.ROUTE_SERIAL)
    S0 = dp.S.clone()
    leaf = synth.root_path(parents[2], 11)
    idx = np.full((4, 8), -1, np.int32); ln = np.zeros(4, np.int32)
    idx[2, :len(leaf)] = leaf[::-1]; ln[2] = len(leaf)                   # reversed: not a chain from a root
    idx[0, :1] = [0]; ln[0] = 1
    dp.path_idx.copy_(torch.from_numpy(idx)); dp.path_len.copy_(torch.from_numpy(ln))
    dp.commit()
    assert dp.status_value() & speca.STATUS_BAD_PATH
    assert torch.equal(dp.S[:, 2], S0[:, 2]) and torch.equal(dp.S[:, 1], S0[:, 1])
    assert not torch.equal(dp.S[:, 0], S0[:, 0])
    dp.status.zero_()
    ln[:] = 0; ln[3] = 9
    dp.path_len.copy_(torch.from_numpy(ln))
    S1 = dp.S.clone()
    dp.commit()
    assert dp.status_value() & speca.STATUS_TOO_DEEP and torch.equal(dp.S, S1)


def test_outputs_stay_inside_their_buffers():
    """Guard bands around o and S: nothing outside the tensors is written."""
    prob = synth.config(3, L=2)
    dp = DevProblem(prob, route=speca.ROUTE_SERIAL)
    n = dp.o.numel()
    big = torch.full((n + 512,), 7.5, device="cuda")
    dp.o = big[256:256 + n].view_as(dp.o)
    dp.verify_tree()
    torch.cuda.synchronize()
    assert torch.all(big[:256] == 7.5) and torch.all(big[-256:] == 7.5)
    ns = dp.S.numel()
    bigS = torch.full((ns + 512,), 7.5, device="cuda")
    bigS[256:256 + ns] = dp.S.flatten()
    dp.S = bigS[256:256 + ns].view_as(dp.S)
    dp.commit()
    torch.cuda.synchronize()
    assert torch.all(bigS[:256] == 7.5) and torch.all(bigS[-256:] == 7.5)
    assert dp.status_value() == 0


def test_accept_matches_oracle_on_many_random_batches():
    rng = np.random.default_rng(123)
    for trial in range(6):
        parents = synth.ragged_tree_batch(rng, 40, 1, 64, 8)
        prob = synth.make_problem(200 + trial, 1, 1, 64, 32, parents, p_match=0.85)
        dp = DevProblem(prob)
        dp.accept()
        pi, pl, nt = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                          prob.root_target_tok, prob.max_depth)
        assert dp.status_value() == 0
        assert np.array_equal(cpu(dp.path_idx), pi) and np.array_equal(cpu(dp.path_len), pl)
        assert np.array_equal(cpu(dp.next_tok), nt)


def test_multi_round_loop_carries_state():
    """verify -> accept -> commit for several rounds with fresh drafts, the oracle carrying its own fp64 state."""
    rng = np.random.default_rng(31)
    L, B, H, dk, dv = 2, 6, 2, 128, 256
    S_ref = None
    S_dev = None
    for rnd in range(4):
        parents = synth.mixed_chain_tree_batch(rng, B, 8, 40, 8)
        prob = synth.make_problem(300 + rnd, L, H, dk, dv, parents, p_match=0.9)
        if S_ref is None:
            S_ref = prob.S0.astype(np.float64)
        dp = DevProblem(prob, route=speca.ROUTE_SERIAL)
        if S_dev is not None:
            dp.S.copy_(S_dev)
        o = dp.verify_tree()
        o_ref = oracle.verify_tree(S_ref, prob.q, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets,
                                   prob.parent)
        assert rel_err(cpu(o), o_ref) <= TOL_FP32 * (rnd + 1)
        dp.accept()
        pi, pl, nt = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                          prob.root_target_tok, prob.max_depth)
        assert np.array_equal(cpu(dp.path_idx), pi) and np.array_equal(cpu(dp.path_len), pl)
        dp.commit()
        S_ref = oracle.commit(S_ref, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets, pi, pl)
        assert rel_err(cpu(dp.S), S_ref) <= TOL_FP32 * (rnd + 1)
        assert dp.status_value() == 0
        S_dev = dp.S.clone()


# ---------------------------------------------------------------------------
# factorised (tensor-core) route: shapes and edge cases of its own
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("d_v", [128, 256])
def test_factorized_edge_cases(d_v):
    rng = np.random.default_rng(900 + d_v)
    forest = np.array([-1, -1, 0, -1, 1, 1, 2, 3, 3, 6], np.int32)       # three roots
    stars = np.array([-1] * 6, np.int32)                                   # "all-root" proposal
    bfs = synth.beam_tree_parent(4, 8, 31, rng)                            # breadth-first node order (not depth-first)
    parents = [np.zeros(0, np.int32), synth.chain_parent(1), forest, stars, bfs, synth.chain_parent(8),
               synth.random_tree_parent(64, 8, 4, rng), synth.random_tree_parent(17, 8, 2, rng),
               synth.random_tree_parent(48, 5, 4, rng), np.zeros(0, np.int32), synth.random_tree_parent(33, 8, 4, rng)]
    prob = synth.make_problem(901 + d_v, 3, 5, 128, d_v, parents, name=f"fact-edges-{d_v}")
    prob.scale = 0.5
    dp, ref = check_verify(prob, speca.ROUTE_FACTORIZED, want_u=True, max_nodes=64)
    # the serial route on the same inputs agrees with the factorised one far inside the bar
    ds = DevProblem(prob, route=speca.ROUTE_SERIAL, want_u=True, max_nodes=64)
    ds.verify_tree()
    assert rel_err(cpu(dp.o), cpu(ds.o)) <= TOL_FP32 and rel_err(cpu(dp.u), cpu(ds.u)) <= TOL_FP32
    # chain entry point on the factorised route (no parent array)
    chains = [synth.chain_parent(n) for n in (8, 1, 5, 7, 8)]
    cp = synth.make_problem(902 + d_v, 2, 3, 128, d_v, chains, name="fact-chains")
    check_verify(cp, speca.ROUTE_FACTORIZED, chain=True, max_nodes=16)


def test_factorized_faults_skip_the_sequence():
    rng = np.random.default_rng(950)
    parents = [synth.random_tree_parent(12, 5, 3, rng) for _ in range(4)]
    prob = synth.make_problem(951, 2, 2, 128, 128, parents)
    good = oracle_verify(prob)
    s1, e1 = int(prob.node_offsets[1]), int(prob.node_offsets[2])
    prob.parent[s1 + 3] = 7
    dp = DevProblem(prob, route=speca.ROUTE_FACTORIZED, max_nodes=16)
    dp.verify_tree(with_depth=False)
    assert dp.status_value() == speca.STATUS_BAD_PARENT
    o = cpu(dp.o)
    assert np.all(np.isnan(o[:, s1:e1]))
    keep = np.r_[0:s1, e1:prob.T]
    assert rel_err(o[:, keep], good[:, keep]) <= TOL_FP32


@pytest.mark.parametrize("d_v", [128, 256])
def test_factorized_key_width_256(d_v):
    """The paper's target shape (d_k = 256): the tensor-core route takes up to 32 nodes per sequence."""
    rng = np.random.default_rng(970 + d_v)
    forest = np.array([-1, -1, 0, -1, 1, 1, 2, 3, 3, 6], np.int32)
    parents = [np.zeros(0, np.int32), synth.chain_parent(1), forest, synth.chain_parent(8),
               synth.random_tree_parent(32, 8, 4, rng), synth.proposal_tree_parent(4, 4, 32, rng),
               synth.random_tree_parent(17, 8, 2, rng), synth.proposal_tree_parent(4, 4, 16, rng),
               synth.random_tree_parent(29, 5, 4, rng)]
    prob = synth.make_problem(971 + d_v, 3, 8, 256, d_v, parents, name=f"fact-dk256-{d_v}")
    dp, ref = check_verify(prob, speca.ROUTE_FACTORIZED, want_u=True, max_nodes=32)
    ds = DevProblem(prob, route=speca.ROUTE_SERIAL, want_u=True, max_nodes=32)
    ds.verify_tree()
    assert rel_err(cpu(dp.o), cpu(ds.o)) <= TOL_FP32 and rel_err(cpu(dp.u), cpu(ds.u)) <= TOL_FP32
    # accept + commit on the same records (commit is the fp32 kernel whatever verified)
    dp.accept()
    pi, pl, _ = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                     prob.root_target_tok, prob.max_depth)
    assert np.array_equal(cpu(dp.path_idx), pi) and np.array_equal(cpu(dp.path_len), pl)
    dp.commit()
    assert rel_err(cpu(dp.S), oracle_commit(prob, pi, pl)) <= TOL_FP32
    # 33 nodes is one too many for this key width: refused when asked for explicitly, serial under AUTO
    big = synth.make_problem(972, 1, 2, 256, d_v, [synth.random_tree_parent(33, 8, 4, rng)])
    with pytest.raises(speca.SpecaError, match="unsupported"):
        DevProblem(big, route=speca.ROUTE_FACTORIZED, max_nodes=33).verify_tree()
    check_verify(big, speca.ROUTE_AUTO, tol=TOL_FP32, max_nodes=33)


def test_factorized_key_width_256_batched_paper_shape():
    """h_v = 8, d_k = d_v = 256, a batch of proposal trees (depth <= 8): every unit against the oracle."""
    rng = np.random.default_rng(980)
    parents = [synth.proposal_tree_parent(4, int(rng.integers(3, 9)), int(rng.integers(8, 33)), rng) for _ in range(24)]
    prob = synth.make_problem(981, 2, 8, 256, 256, parents, name="paper-shape-batch")
    check_verify(prob, speca.ROUTE_AUTO, max_nodes=32)


def test_round_is_cuda_graph_capturable():
    """No entry point allocates or synchronises, so a whole round can be captured once and replayed."""
    rng = np.random.default_rng(990)
    prob = synth.make_problem(991, 2, 4, 128, 256, synth.ragged_tree_batch(rng, 4, 4, 40, 8))
    eager = DevProblem(prob, route=speca.ROUTE_AUTO, max_nodes=64)
    eager.verify_tree(); eager.accept(); eager.commit()
    assert eager.status_value() == 0
    dp = DevProblem(prob, route=speca.ROUTE_AUTO, max_nodes=64)
    S0 = dp.S.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        dp.verify_tree(); dp.accept(); dp.commit()                 # warm-up outside the capture (first-call attributes)
        dp.S.copy_(S0)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            dp.verify_tree(); dp.accept(); dp.commit()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        dp.S.copy_(S0)
        dp.o.fill_(float("nan"))
        g.replay()
        assert dp.status_value() == 0
        assert torch.equal(dp.o, eager.o) and torch.equal(dp.S, eager.S)
        assert torch.equal(dp.path_idx, eager.path_idx) and torch.equal(dp.path_len, eager.path_len)


@pytest.mark.parametrize("route", ROUTES)
def test_deltanet_records_are_the_alpha_one_case(route):
    """A DeltaNet layer keeps (k, v, beta) and has no decay: the same entry points with alpha = 1
    (Section 5.1, remark on other layer types).  Verify, commit and the fused call against the oracle."""
    rng = np.random.default_rng(995)
    p1 = synth.make_problem(996, 2, 4, 128, 128, synth.ragged_tree_batch(rng, 4, 4, 30, 8))
    p2 = synth.make_problem(997, 2, 4, 128, 128, synth.ragged_tree_batch(rng, 4, 4, 30, 8))
    p1.alpha[:] = 1.0
    p2.alpha[:] = 1.0
    d1, _ = check_verify(p1, route, want_u=True, max_nodes=64)
    d1.accept()
    pi, pl, _ = oracle.greedy_accept(p1.node_offsets, p1.parent, p1.draft_tok, p1.target_tok, p1.root_target_tok, 8)
    d2 = DevProblem(p2, route=route, want_u=True, max_nodes=64)
    S = d1.S.clone()
    prev = dict(k=d1.k, v=d1.v, alpha=d1.alpha, beta=d1.beta, u=d1.u, node_offsets=d1.node_offsets, total_nodes=d1.T,
                parent=d1.parent)
    speca.commit_verify_tree(d2.dims, S, prev, d1.path_idx, d1.path_len, d2.q, d2.k, d2.v, d2.alpha, d2.beta,
                             d2.node_offsets, d2.T, d2.parent, None, d2.o, d2.u, d2.ws, d2.status)
    assert d2.status_value() == 0
    S_ref = oracle_commit(p1, pi, pl)
    o_ref = oracle.verify_tree(S_ref, p2.q, p2.k, p2.v, p2.alpha, p2.beta, p2.node_offsets, p2.parent)
    assert rel_err(cpu(S), S_ref) <= tol_for(route) and rel_err(cpu(d2.o), o_ref) <= tol_for(route)
    d1.commit()
    assert rel_err(cpu(d1.S), S_ref) <= TOL_FP32


@pytest.mark.parametrize("route", ROUTES)
def test_rule_without_erase(route):
    """GLA-style records (key, value, gate; no delta-rule read-out): dims.rule = GATED_NO_ERASE on decode,
    verify, commit and the fused call, against the oracle set to the same rule."""
    rng = np.random.default_rng(1001)
    p1 = synth.make_problem(1002, 2, 4, 128, 256, synth.ragged_tree_batch(rng, 4, 4, 40, 8))
    p2 = synth.make_problem(1003, 2, 4, 128, 256, synth.ragged_tree_batch(rng, 4, 4, 40, 8))
    R = speca.RULE_GATED_NO_ERASE
    try:
        oracle.set_rule(oracle.RULE_GATED_NO_ERASE)
        o1_ref = oracle_verify(p1)
        pi, pl, _ = oracle.greedy_accept(p1.node_offsets, p1.parent, p1.draft_tok, p1.target_tok, p1.root_target_tok, 8)
        S_ref = oracle_commit(p1, pi, pl)
        o2_ref = oracle.verify_tree(S_ref, p2.q, p2.k, p2.v, p2.alpha, p2.beta, p2.node_offsets, p2.parent)
        q1, k1, v1, a1, b1 = synth.draw_records(rng, p1.L, p1.B, p1.H, p1.d_k, p1.d_v)
        Sd_ref, od_ref = oracle.decode_step(p1.S0, q1, k1, v1, a1, b1)
    finally:
        oracle.set_rule(oracle.RULE_GATED_DELTA)
    d1 = DevProblem(p1, route=route, want_u=True, max_nodes=64, rule=R)
    d1.verify_tree()
    assert d1.status_value() == 0 and rel_err(cpu(d1.o), o1_ref) <= tol_for(route)
    d1.accept()
    d2 = DevProblem(p2, route=route, want_u=True, max_nodes=64, rule=R)
    S = d1.S.clone()
    prev = dict(k=d1.k, v=d1.v, alpha=d1.alpha, beta=d1.beta, u=d1.u, node_offsets=d1.node_offsets, total_nodes=d1.T,
                parent=d1.parent)
    speca.commit_verify_tree(d2.dims, S, prev, d1.path_idx, d1.path_len, d2.q, d2.k, d2.v, d2.alpha, d2.beta,
                             d2.node_offsets, d2.T, d2.parent, None, d2.o, d2.u, d2.ws, d2.status)
    assert d2.status_value() == 0
    assert rel_err(cpu(S), S_ref) <= tol_for(route) and rel_err(cpu(d2.o), o2_ref) <= tol_for(route)
    d1.commit()
    assert rel_err(cpu(d1.S), S_ref) <= TOL_FP32
    from gpu_util import bf16_dev
    Sd = torch.from_numpy(p1.S0).cuda()
    od = torch.empty(p1.L, p1.B, p1.H, p1.d_v, device="cuda")
    speca.decode_step(speca.Dims(p1.L, p1.B, p1.H, p1.d_k, p1.d_v, rule=R), Sd, bf16_dev(q1), bf16_dev(k1), bf16_dev(v1),
                      torch.from_numpy(a1).cuda(), torch.from_numpy(b1).cuda(), od)
    assert rel_err(cpu(Sd), Sd_ref) <= TOL_FP32 and rel_err(cpu(od), od_ref) <= TOL_FP32


@pytest.mark.parametrize("d_k,d_v", [(128, 128), (128, 256), (256, 128), (256, 256)])
def test_factorized_deep_trees(d_k, d_v):
    """Trees 9 to 16 levels deep (the paper's top-2 proposal shapes) on the tensor-core route: up to 32 nodes."""
    rng = np.random.default_rng(1100 + d_k + d_v)
    parents = [synth.proposal_tree_parent(2, 12, 16, rng), synth.proposal_tree_parent(2, 24, 32, rng),
               synth.proposal_tree_parent(4, 12, 16, rng), synth.chain_parent(16), np.zeros(0, np.int32),
               synth.random_tree_parent(32, 16, 3, rng), synth.chain_parent(1), synth.random_tree_parent(20, 5, 3, rng),
               synth.chain_parent(9)]
    prob = synth.make_problem(1101 + d_k + d_v, 2, 4, d_k, d_v, parents, max_depth=16, name=f"deep-{d_k}x{d_v}")
    assert int(prob.depth.max()) == 16
    dp, ref = check_verify(prob, speca.ROUTE_FACTORIZED, want_u=True, max_nodes=32)
    ds = DevProblem(prob, route=speca.ROUTE_SERIAL, want_u=True, max_nodes=32)
    ds.verify_tree()
    assert rel_err(cpu(dp.o), cpu(ds.o)) <= TOL_FP32 and rel_err(cpu(dp.u), cpu(ds.u)) <= TOL_FP32
    # paths up to 16 nodes long: accept and commit (fp32 kernel)
    dp.accept()
    pi, pl, _ = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                     prob.root_target_tok, prob.max_depth)
    assert np.array_equal(cpu(dp.path_idx), pi) and np.array_equal(cpu(dp.path_len), pl)
    dp.commit()
    assert rel_err(cpu(dp.S), oracle_commit(prob, pi, pl)) <= TOL_FP32
    # 33 nodes at this depth: d_k = 128 goes to the effective-query kernel, d_k = 256 is outside every tensor-core route
    big = synth.make_problem(1102, 1, 2, d_k, d_v, [synth.random_tree_parent(33, 12, 3, rng)], max_depth=16)
    if d_k == 128:
        check_verify(big, speca.ROUTE_FACTORIZED, max_nodes=33)
    else:
        with pytest.raises(speca.SpecaError, match="unsupported"):
            DevProblem(big, route=speca.ROUTE_FACTORIZED, max_nodes=33).verify_tree()
    check_verify(big, speca.ROUTE_AUTO, tol=TOL_FP32, max_nodes=33)


def test_fused_call_with_deep_trees_takes_the_two_kernel_path():
    rng = np.random.default_rng(1200)
    mk = lambda seed: synth.make_problem(seed, 2, 4, 128, 256, [synth.proposal_tree_parent(2, 12, 16, rng), synth.chain_parent(12),
                                                                 synth.random_tree_parent(30, 14, 3, rng)], max_depth=16)
    p1, p2 = mk(1201), mk(1202)
    paths = [synth.root_path(p1.parent[int(p1.node_offsets[b]):int(p1.node_offsets[b + 1])],
                             int(np.argmax(p1.depth[int(p1.node_offsets[b]):int(p1.node_offsets[b + 1])]))) for b in range(3)]
    idx = np.full((3, 16), -1, np.int32); ln = np.zeros(3, np.int32)
    for b, pth in enumerate(paths):
        idx[b, :len(pth)] = pth; ln[b] = len(pth)
    p1.path_idx, p1.path_len = idx, ln
    d1 = DevProblem(p1, route=speca.ROUTE_AUTO, want_u=True, max_nodes=32)
    d1.verify_tree()
    d2 = DevProblem(p2, route=speca.ROUTE_AUTO, want_u=True, max_nodes=32)
    S = d1.S.clone()
    prev = dict(k=d1.k, v=d1.v, alpha=d1.alpha, beta=d1.beta, u=d1.u, node_offsets=d1.node_offsets, total_nodes=d1.T,
                parent=d1.parent)
    speca.commit_verify_tree(d2.dims, S, prev, d1.path_idx, d1.path_len, d2.q, d2.k, d2.v, d2.alpha, d2.beta,
                             d2.node_offsets, d2.T, d2.parent, None, d2.o, d2.u, d2.ws, d2.status)
    assert d2.status_value() == 0
    S_ref = oracle_commit(p1, idx, ln)
    o_ref = oracle.verify_tree(S_ref, p2.q, p2.k, p2.v, p2.alpha, p2.beta, p2.node_offsets, p2.parent)
    assert rel_err(cpu(S), S_ref) <= TOL_FP32 and rel_err(cpu(d2.o), o_ref) <= TOL_FP32


def test_expired_wait_is_reported_and_the_context_stays_usable():
    """Failure detection: every device-side wait is bounded.  With the library's test hook one CTA's first
    state slice is never requested; its waits run out (2 s), the kernel returns, the status word carries
    TIMEOUT, and the next call on the same context works."""
    rng = np.random.default_rng(1300)
    prob = synth.make_problem(1301, 2, 4, 128, 128, synth.ragged_tree_batch(rng, 3, 4, 20, 8))
    dp = DevProblem(prob, route=speca.ROUTE_FACTORIZED, max_nodes=64)
    hook = speca.lib().speca_test_withhold_first_load        # test-only symbol, not in the public header
    hook.argtypes, hook.restype = [ctypes.c_int], None
    hook(1)
    try:
        dp.verify_tree()
        assert dp.status_value() & speca.STATUS_TIMEOUT
    finally:
        hook(0)
    dp.status.zero_()
    dp.o.fill_(float("nan"))
    dp.verify_tree()
    assert dp.status_value() == 0
    assert rel_err(cpu(dp.o), oracle_verify(prob)) <= TOL_FP32


@pytest.mark.parametrize("route", [speca.ROUTE_SERIAL, speca.ROUTE_AUTO])
def test_chain_longer_than_max_depth_is_a_fault_on_every_route(route):
    """A chain of n nodes is n levels deep: the chain entry point reports TOO_DEEP and skips the sequence whatever
    kernel verifies it."""
    prob = synth.make_problem(1400, 1, 2, 128, 128, [synth.chain_parent(6), synth.chain_parent(12)], max_depth=16)
    good = oracle_verify(prob)
    dp = DevProblem(prob, route=route, max_nodes=16)
    dp.dims.max_depth = 8
    dp.verify_chain()
    assert dp.status_value() == speca.STATUS_TOO_DEEP
    o = cpu(dp.o)
    assert np.all(np.isnan(o[:, 6:]))
    assert rel_err(o[:, :6], good[:, :6]) <= TOL_FP32
