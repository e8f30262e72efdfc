"""Commit of long accepted paths (Section 5.1, Eq. 3; Section 5.2): paths of four to eight nodes are committed
by the tensor-core kernel, shorter and longer ones token by token.  Every length, both kernels in one batch,
against the fp64 oracle's token-by-token recurrence."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth
from gpu_util import DevProblem, TOL_FP32, max_err_over_max, oracle_commit, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["long-path kernel", "size rule"])
def long_kernel_for_every_batch(request):
    """By default only throughput-sized batches go to the tensor-core kernel; the test-only switch (not in the
    public header) makes these small batches take it.  Every test runs both ways."""
    hook = speca.lib().speca_test_commit_long_min_tiles
    hook(0 if request.param == "long-path kernel" else -1)
    yield
    hook(-1)


def cpu(t):
    return t.detach().cpu().numpy()


def deep_parents(n_seq, rng, n_nodes=28, max_depth=8):
    """Random trees that each contain a root path of max_depth nodes: a spine 0..max_depth-1, the rest at random."""
    out = []
    for _ in range(n_seq):
        p = synth.random_tree_parent(n_nodes, max_depth, 3, rng)
        p[:max_depth] = np.arange(-1, max_depth - 1)
        out.append(p)
    return out


def set_paths(dp, prob, paths):
    idx = np.full((prob.B, prob.max_depth), -1, np.int32)
    ln = np.zeros(prob.B, np.int32)
    for b, path in enumerate(paths):
        idx[b, :len(path)] = path
        ln[b] = len(path)
    dp.path_idx.copy_(torch.from_numpy(idx))
    dp.path_len.copy_(torch.from_numpy(ln))
    return idx, ln


def paths_of_lengths(prob, parents, lengths, rng):
    """For each sequence a root path of the wanted length: the path of a random node at that depth."""
    paths = []
    for b, want in enumerate(lengths):
        if want == 0:
            paths.append([])
            continue
        depth = synth.depth_of(parents[b])
        cand = np.flatnonzero(depth == want)
        assert cand.size, "the spine guarantees a node at every depth"
        paths.append(synth.root_path(parents[b], int(rng.choice(cand))))
    return paths


@pytest.mark.parametrize("d_k,d_v", [(64, 64), (64, 128), (128, 96), (128, 128), (128, 256), (256, 256)])
@pytest.mark.parametrize("state_std", [0.02, 4.0])
def test_every_path_length_in_one_batch(d_k, d_v, state_std):
    rng = np.random.default_rng(300 + d_k + d_v)
    lengths = [0, 1, 2, 3, 4, 5, 6, 7, 8, 8, 4, 5, 0, 6]
    parents = deep_parents(len(lengths), rng)
    prob = synth.make_problem(301, 2, 3, d_k, d_v, parents, state_std=state_std)
    dp = DevProblem(prob)
    idx, ln = set_paths(dp, prob, paths_of_lengths(prob, parents, lengths, rng))
    S0 = dp.S.clone()
    dp.commit()
    assert dp.status_value() == 0
    ref = oracle_commit(prob, idx, ln)
    S = cpu(dp.S)
    for b, want in enumerate(lengths):
        if want == 0:
            assert torch.equal(dp.S[:, b], S0[:, b]), "an empty path leaves the state bitwise untouched"
        else:
            e = rel_err(S[:, b], ref[:, b])
            assert e <= TOL_FP32, f"path of {want} nodes: state error {e:.3e}"
    print(f"d_k={d_k} d_v={d_v} std={state_std}: state err {rel_err(S, ref):.2e} "
          f"(max|x-r|/max|r| {max_err_over_max(S, ref):.2e})")


def test_long_paths_without_the_parent_check_and_on_chains():
    prob = synth.make_problem(310, 3, 4, 128, 256, [synth.chain_parent(8) for _ in range(9)])
    dp = DevProblem(prob)
    idx, ln = set_paths(dp, prob, [list(range(n)) for n in (8, 7, 6, 5, 4, 3, 2, 1, 8)])
    dp.commit(check_parent=False)
    assert dp.status_value() == 0
    assert rel_err(cpu(dp.S), oracle_commit(prob, idx, ln)) <= TOL_FP32


def test_long_path_equals_repeated_decode_steps():
    """A committed chain of eight is eight decode steps on the same records (Section 2.2)."""
    prob = synth.make_problem(311, 2, 2, 128, 128, [synth.chain_parent(8), synth.chain_parent(8)])
    dp = DevProblem(prob)
    set_paths(dp, prob, [list(range(8)), list(range(6))])
    dp.commit()
    S = torch.from_numpy(prob.S0).cuda()
    d1 = speca.Dims(prob.L, prob.B, prob.H, prob.d_k, prob.d_v)
    o = torch.empty(prob.L, prob.B, prob.H, prob.d_v, device="cuda")
    for step in range(8):
        take = [int(prob.node_offsets[b]) + step for b in range(prob.B)]
        rec = lambda x: x[:, take].contiguous()
        S_before = S.clone()
        speca.decode_step(d1, S, rec(dp.q), rec(dp.k), rec(dp.v), rec(dp.alpha), rec(dp.beta), o)
        if step >= 6:
            S[:, 1] = S_before[:, 1]                       # the second sequence accepted six nodes only
    assert rel_err(cpu(dp.S), cpu(S)) <= TOL_FP32


def test_faults_on_long_paths_leave_the_state_untouched():
    rng = np.random.default_rng(320)
    parents = deep_parents(5, rng)
    prob = synth.make_problem(321, 2, 2, 128, 128, parents)
    dp = DevProblem(prob)
    paths = paths_of_lengths(prob, parents, [6, 6, 5, 2, 8], rng)
    paths[1] = paths[1][::-1]                               # not a chain from a root
    paths[2] = paths[2][:-1] + [99]                         # node index outside the sequence
    idx, ln = set_paths(dp, prob, paths)
    S0 = dp.S.clone()
    dp.commit()
    assert dp.status_value() & speca.STATUS_BAD_PATH
    assert torch.equal(dp.S[:, 1], S0[:, 1]) and torch.equal(dp.S[:, 2], S0[:, 2])
    good = [0, 3, 4]
    ln_ok = ln.copy(); ln_ok[[1, 2]] = 0
    ref = oracle_commit(prob, idx, ln_ok)
    assert rel_err(cpu(dp.S)[:, good], ref[:, good]) <= TOL_FP32


def test_paths_longer_than_eight_and_wide_path_rows():
    """max_depth = 16: rows of path_idx are 16 wide; nine nodes and more stay with the token-by-token kernel."""
    parents = [synth.chain_parent(14), synth.chain_parent(14), synth.chain_parent(14), synth.chain_parent(5)]
    prob = synth.make_problem(330, 2, 2, 128, 128, parents, max_depth=16)
    dp = DevProblem(prob)
    idx, ln = set_paths(dp, prob, [list(range(12)), list(range(8)), list(range(9)), list(range(4))])
    dp.commit()
    assert dp.status_value() == 0
    assert rel_err(cpu(dp.S), oracle_commit(prob, idx, ln)) <= TOL_FP32


def test_rule_without_erase_on_long_paths():
    rng = np.random.default_rng(340)
    parents = deep_parents(6, rng)
    prob = synth.make_problem(341, 2, 3, 128, 256, parents)
    dp = DevProblem(prob, rule=speca.RULE_GATED_NO_ERASE)
    idx, ln = set_paths(dp, prob, paths_of_lengths(prob, parents, [8, 4, 3, 6, 0, 5], rng))
    dp.commit()
    assert dp.status_value() == 0
    try:
        oracle.set_rule(oracle.RULE_GATED_NO_ERASE)
        ref = oracle_commit(prob, idx, ln)
    finally:
        oracle.set_rule(oracle.RULE_GATED_DELTA)
    assert rel_err(cpu(dp.S), ref) <= TOL_FP32


def test_small_batch_takes_single_tiles_and_large_batch_whole_units():
    """The rows a warp takes per work item depend on the batch: both ends give the same state."""
    for L, B in ((1, 1), (4, 40)):
        prob = synth.make_problem(350 + B, L, 16, 128, 256, [synth.chain_parent(8) for _ in range(B)])
        dp = DevProblem(prob)
        idx, ln = set_paths(dp, prob, [list(range(8 - (b % 3))) for b in range(B)])
        dp.commit()
        assert dp.status_value() == 0
        assert rel_err(cpu(dp.S), oracle_commit(prob, idx, ln)) <= TOL_FP32


def test_commit_with_long_paths_is_cuda_graph_capturable():
    """Both commit launches go into a captured graph; a replay gives the eager state bit for bit."""
    prob = synth.make_problem(360, 2, 4, 128, 256, [synth.chain_parent(8) for _ in range(6)])
    paths = [list(range(n)) for n in (8, 2, 5, 0, 7, 3)]
    eager = DevProblem(prob)
    set_paths(eager, prob, paths)
    eager.commit()
    assert eager.status_value() == 0
    dp = DevProblem(prob)
    set_paths(dp, prob, paths)
    S0 = dp.S.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        dp.commit()                                        # warm-up outside the capture (first-call device queries)
        dp.S.copy_(S0)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            dp.commit()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        dp.S.copy_(S0)
        g.replay()
        assert dp.status_value() == 0
        assert torch.equal(dp.S, eager.S)


def test_random_batches_of_paths():
    """Seeded random shapes, trees and accepted paths (every length 0..8 mixed), 12 batches."""
    rng = np.random.default_rng(370)
    for it in range(12):
        d_k = int(rng.choice([64, 128]))
        d_v = int(rng.choice([64, 128, 256]))
        B = int(rng.integers(1, 9))
        parents = deep_parents(B, rng, n_nodes=int(rng.integers(8, 40)))
        prob = synth.make_problem(371 + it, int(rng.integers(1, 4)), int(rng.integers(1, 5)), d_k, d_v, parents,
                                  state_std=float(rng.choice([0.02, 0.5])))
        dp = DevProblem(prob)
        lengths = [int(rng.integers(0, 9)) for _ in range(B)]
        idx, ln = set_paths(dp, prob, paths_of_lengths(prob, parents, lengths, rng))
        dp.commit(check_parent=bool(it & 1))
        assert dp.status_value() == 0
        e = rel_err(cpu(dp.S), oracle_commit(prob, idx, ln))
        assert e <= TOL_FP32, f"batch {it} (d_k={d_k}, d_v={d_v}, lengths {lengths}): state error {e:.3e}"
