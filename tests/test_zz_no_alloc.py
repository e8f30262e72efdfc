"""speca_verify_tree_noalloc: the verify entry point for callers that cannot allocate.

Some users of the library run where device allocation is not an option: a serving loop
with a memory pool frozen at start-up, a plug-in that receives tensors but no allocator,
a latency-critical stream that must never hit the device-wide synchronisation of
cudaMalloc.  For them the library carries its own fixed scratch array.  This test calls
that entry point through the C ABI twice in a row (the second call finds the first
call's leftovers in the array) and checks both results against the ordinary entry point
fed with a caller-allocated workspace, and against the fp64 oracle.

Collected last on purpose, so that a run stopping at the first failure has already run
every other test; it must also pass alone in a fresh process.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth
from gpu_util import DevProblem, TOL_FP32, oracle_verify, rel_err


def _problem(seed, sizes):
    rng = np.random.default_rng(seed)
    parents = [synth.random_tree_parent(n, 8, 4, rng) if n > 1 else synth.chain_parent(n) for n in sizes]
    return synth.make_problem(seed, 2, 4, 128, 128, parents, state_std=0.3, p_match=0.8)


@pytest.mark.gpu
@pytest.mark.parametrize("route", [speca.ROUTE_SERIAL, speca.ROUTE_AUTO])
def test_noalloc_matches_workspace_entry_point_twice_in_a_row(route):
    # two different problems back to back: the second call must not be disturbed by what the
    # first one left in the shared scratch (a longer batch first, then a shorter one)
    for seed, sizes in [(41, [33, 8, 1, 64, 17, 5]), (42, [12, 40, 3])]:
        prob = _problem(seed, sizes)
        ref = DevProblem(prob, route=route, want_u=True, max_nodes=64)
        ref.verify_tree()
        assert ref.status_value() == 0
        dp = DevProblem(prob, route=route, want_u=True, max_nodes=64)
        speca.verify_tree_noalloc(dp.dims, dp.S, dp.q, dp.k, dp.v, dp.alpha, dp.beta, dp.node_offsets, dp.T,
                                  dp.parent, dp.depth, dp.o, dp.u, dp.status)
        assert dp.status_value() == 0
        # same kernels, same inputs: the tolerance of the other parity tests is ample
        assert rel_err(dp.o.cpu().numpy(), ref.o.cpu().numpy()) <= TOL_FP32
        assert rel_err(dp.u.cpu().numpy(), ref.u.cpu().numpy()) <= TOL_FP32
        assert torch.equal(dp.S, ref.S)
        # and an error common to both entry points would show against the oracle
        assert rel_err(dp.o.cpu().numpy(), oracle_verify(prob)) <= TOL_FP32


@pytest.mark.gpu
def test_noalloc_rejects_problems_beyond_its_scratch():
    prob = _problem(43, [4, 4])
    dp = DevProblem(prob, max_nodes=64)
    big = speca.Dims(1, speca.NOALLOC_MAX_BATCH + 1, 1, 128, 128)
    d = big.c()
    rc = speca.lib().speca_verify_tree_noalloc(ctypes.byref(d), *([ctypes.c_void_p(dp.S.data_ptr())] * 7), 8,
                                               *([ctypes.c_void_p(dp.S.data_ptr())] * 5),
                                               ctypes.c_void_p(dp.status.data_ptr()), None)
    assert rc == -7 and b"built-in scratch" in speca.lib().speca_strerror(rc)
    d = dp.dims.c()
    rc = speca.lib().speca_verify_tree_noalloc(ctypes.byref(d), *([ctypes.c_void_p(dp.S.data_ptr())] * 7),
                                               speca.NOALLOC_MAX_NODES + 1,
                                               *([ctypes.c_void_p(dp.S.data_ptr())] * 5),
                                               ctypes.c_void_p(dp.status.data_ptr()), None)
    assert rc == -7
    assert dp.status_value() == 0
