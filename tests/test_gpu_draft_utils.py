"""GPU parity of the draft-side integer utilities (tree-mask converter, confidence-guided pruning): bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth

pytestmark = pytest.mark.gpu
t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()


def mask_of(parents, N):
    m = np.zeros((len(parents), N, N), np.uint8)
    for b, par in enumerate(parents):
        for i in range(len(par)):
            for a in synth.root_path(par, i):
                m[b, i, a] = 1
    return m


def batch(rng, B, lo, hi):
    parents = [synth.random_tree_parent(int(rng.integers(lo, hi + 1)), 8, 4, rng) for _ in range(B)]
    parents[B // 2] = np.zeros(0, np.int32)
    parents[0] = np.array([-1, -1, 0, -1, 1], np.int32)
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    return parents, offs


def test_tree_mask_to_parent():
    rng = np.random.default_rng(61)
    parents, offs = batch(rng, 40, 1, 64)
    mask = mask_of(parents, 64)
    T = int(offs[-1])
    par = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    speca.tree_mask_to_parent(t(mask), t(offs), par, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(par.cpu().numpy(), oracle.tree_mask_to_parent(mask, offs))
    assert np.array_equal(par.cpu().numpy(), np.concatenate(parents))
    # a mask that is not a tree mask (node 3 of sequence 1 sees node 1 but not node 1's parent)
    bad = mask.copy()
    p1 = parents[1]
    deep = int(np.argmax(synth.depth_of(p1)))
    if synth.depth_of(p1)[deep] >= 3:
        bad[1, deep, synth.root_path(p1, deep)[0]] = 0
        par.fill_(-7)
        speca.tree_mask_to_parent(t(bad), t(offs), par, status)
        torch.cuda.synchronize()
        assert int(status.item()) == speca.STATUS_BAD_PARENT
        got = par.cpu().numpy()
        assert np.all(got[offs[1]:offs[2]] == -7)
        keep = np.r_[0:offs[1], offs[2]:T]
        assert np.array_equal(got[keep], np.concatenate(parents)[keep])


@pytest.mark.parametrize("tau,budget", [(0.5, 64), (1.25, 6), (3.0, 16), (10.0, 3), (0.0, 1), (2.0, 0)])
def test_prune_tree(tau, budget):
    rng = np.random.default_rng(62)
    parents, offs = batch(rng, 50, 1, 64)
    parent = np.concatenate(parents).astype(np.int32)
    T = int(offs[-1])
    # realistic scores: log-softmax-like values in fp32 (ties are rare), plus a block of exact ties
    logp = np.log(rng.uniform(0.02, 1.0, T)).astype(np.float32)
    logp[offs[3]:offs[4]] = -0.5
    oo = torch.zeros(len(parents) + 1, dtype=torch.int32, device="cuda")
    op = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    oi = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    speca.prune_tree(64, tau, budget, t(offs), t(parent), t(logp), oo, op, oi, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ro, rp, ri = oracle.prune_tree(offs, parent, logp, tau, budget)
    assert np.array_equal(oo.cpu().numpy(), ro)
    n = int(ro[-1])
    assert np.array_equal(op.cpu().numpy()[:n], rp) and np.array_equal(oi.cpu().numpy()[:n], ri)
    # the pruned topology is a valid input of the verification path
    assert np.all(rp < np.arange(n) - ro[np.searchsorted(ro, np.arange(n), side="right") - 1]) or n == 0


def test_stochastic_accept_matches_the_walk():
    """speca_stochastic_accept against the oracle's walk: paths and lengths bit-exact, over many batches."""
    rng = np.random.default_rng(63)
    for trial in range(6):
        parents, offs = batch(rng, 48, 1, 64)
        if trial == 0:
            parents[1] = synth.chain_parent(8)
            parents[2] = synth.chain_parent(1)
            offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
        parent = np.concatenate(parents).astype(np.int32)
        T = int(offs[-1])
        p_draft = rng.uniform(0.02, 1.0, T).astype(np.float32)
        # ratios p/q on both sides of one, so that paths of every length occur; some exact ties u * q == p
        p_target = (p_draft * rng.choice([0.25, 0.5, 1.0, 2.0], T)).astype(np.float32)
        uniform = rng.random(T, dtype=np.float32)
        ties = rng.random(T) < 0.05
        uniform[ties] = (p_target[ties] / p_draft[ties]).astype(np.float32)
        uniform = np.minimum(uniform, np.float32(0.99999994))
        B = len(parents)
        pidx = torch.full((B, 8), -9, dtype=torch.int32, device="cuda")
        plen = torch.full((B,), -9, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        speca.stochastic_accept(B, 8, t(offs), t(parent), t(p_target), t(p_draft), t(uniform), pidx, plen, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        pi, pl = oracle.stochastic_accept(offs, parent, p_target, p_draft, uniform, 8)
        assert np.array_equal(plen.cpu().numpy(), pl)
        assert np.array_equal(pidx.cpu().numpy(), pi)
        assert pl.max() >= 3 and (pl == 0).any()


def test_stochastic_accept_reports_bad_topology_and_accepts_nothing_there():
    parents = [synth.chain_parent(4), np.array([-1, 1, 0], np.int32), synth.chain_parent(3)]
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    parent = np.concatenate(parents).astype(np.int32)
    T = int(offs[-1])
    one = torch.ones(T, device="cuda")
    zero = torch.zeros(T, device="cuda")
    pidx = torch.full((3, 8), -9, dtype=torch.int32, device="cuda")
    plen = torch.full((3,), -9, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    speca.stochastic_accept(3, 8, t(offs), t(parent), one, one, zero, pidx, plen, status)
    torch.cuda.synchronize()
    assert int(status.item()) & speca.STATUS_BAD_PARENT
    assert plen.cpu().tolist() == [4, 0, 3]
    assert pidx.cpu()[0].tolist() == [0, 1, 2, 3, -1, -1, -1, -1] and pidx.cpu()[1].tolist() == [-1] * 8
    # a chain longer than max_depth is reported, not truncated
    status.zero_()
    speca.stochastic_accept(3, 3, t(offs), t(parent), one, one, zero, pidx[:, :3].contiguous(), plen, status)
    torch.cuda.synchronize()
    assert int(status.item()) & speca.STATUS_TOO_DEEP and plen.cpu().tolist()[0] == 0


def test_chain_decompose_matches_the_definition():
    """speca_chain_decompose against the oracle: chain heads and chain counts bit-exact."""
    rng = np.random.default_rng(64)
    parents, offs = batch(rng, 64, 1, 64)
    parents[3] = synth.chain_parent(8)
    parents[4] = synth.proposal_tree_parent(2, 14, 30, rng, 16)
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    parent = np.concatenate(parents).astype(np.int32)
    T, B = int(offs[-1]), len(parents)
    head = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    speca.chain_decompose(64, t(offs), t(parent), head, cnt, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    h_ref, c_ref = oracle.chain_decompose(offs, parent)
    assert np.array_equal(head.cpu().numpy(), h_ref) and np.array_equal(cnt.cpu().numpy(), c_ref)
    # bad topology: reported, zero chains, entries untouched; the neighbours are still decomposed
    parents = [synth.chain_parent(3), np.array([-1, 1], np.int32), np.array([-1, 0, 0], np.int32)]
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    head = torch.full((8,), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((3,), -7, dtype=torch.int32, device="cuda")
    speca.chain_decompose(64, t(offs), t(np.concatenate(parents).astype(np.int32)), head, cnt, status)
    torch.cuda.synchronize()
    assert int(status.item()) & speca.STATUS_BAD_PARENT
    assert cnt.cpu().tolist() == [1, 0, 2] and head.cpu().tolist() == [0, 0, 0, -7, -7, 0, 0, 2]
