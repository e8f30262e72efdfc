"""GPU parity of the convolution-state commit (bit-exact: 16-bit patterns are moved, not computed)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth

pytestmark = pytest.mark.gpu


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bits_of(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("L,W,ch", [(1, 3, 8), (3, 3, 6144), (2, 1, 64), (2, 8, 200)])
def test_conv_commit_matches_oracle(L, W, ch):
    rng = np.random.default_rng(L * 100 + W * 10 + ch)
    parents = [synth.random_tree_parent(12, 8, 3, rng), synth.chain_parent(8), np.zeros(0, np.int32),
               synth.chain_parent(1), synth.random_tree_parent(30, 8, 4, rng), synth.chain_parent(5)]
    B = len(parents)
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    T = int(offs[-1])
    C = rng.integers(0, 65536, (L, B, W, ch), dtype=np.uint16)
    x = rng.integers(0, 65536, (L, T, ch), dtype=np.uint16)
    # paths: deepest leaf, full chain, nothing, single node, a short path, nothing accepted
    paths = [synth.root_path(parents[0], int(np.argmax(synth.depth_of(parents[0])))), list(range(8)), [], [0],
             synth.root_path(parents[4], 29)[:2], []]
    pidx = np.full((B, 8), -1, np.int32); plen = np.zeros(B, np.int32)
    for b, p in enumerate(paths):
        pidx[b, :len(p)] = p; plen[b] = len(p)
    Cd, xd = dev_bf16(C), dev_bf16(x)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t = lambda a: torch.from_numpy(a).cuda()
    speca.commit_conv(Cd, xd, t(offs), T, t(pidx), t(plen), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(bits_of(Cd), oracle.commit_conv(C, x, offs, pidx, plen))


def test_conv_commit_bad_path_skips_the_sequence():
    L, W, ch = 2, 3, 64
    rng = np.random.default_rng(5)
    offs = np.array([0, 4, 9], np.int32)
    C = rng.integers(0, 65536, (L, 2, W, ch), dtype=np.uint16)
    x = rng.integers(0, 65536, (L, 9, ch), dtype=np.uint16)
    pidx = np.full((2, 8), -1, np.int32); pidx[0, :2] = [0, 7]; pidx[1, :3] = [0, 1, 2]       # 7 is outside sequence 0
    plen = np.array([2, 3], np.int32)
    Cd = dev_bf16(C)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t = lambda a: torch.from_numpy(a).cuda()
    speca.commit_conv(Cd, dev_bf16(x), t(offs), 9, t(pidx), t(plen), status)
    torch.cuda.synchronize()
    assert int(status.item()) == speca.STATUS_BAD_PATH
    good = plen.copy(); good[0] = 0
    assert np.array_equal(bits_of(Cd), oracle.commit_conv(C, x, offs, pidx, good))
