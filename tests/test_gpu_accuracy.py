"""Accuracy of the tensor-core routes whatever the magnitude of the state.

The tensor core reads fp32 operands as TF32 (top 19 bits).  The default routes split both operands into a TF32
head and its exact remainder, so their outputs must sit at the fp32 bar (gpu_util.TOL_FP32) at any state scale,
on a state that happens to be exact in TF32, and after many carried rounds; the single-pass route (ROUTE_TF32)
is only held to the 2e-3 bar, which it reaches as the state grows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth
from gpu_util import DevProblem, TOL, TOL_FP32, max_err_over_max, oracle_commit, oracle_verify, rel_err

pytestmark = pytest.mark.gpu

ACCURATE = [speca.ROUTE_FACTORIZED, speca.ROUTE_EFFECTIVE, speca.ROUTE_AUTO]


def cpu(t):
    return t.detach().cpu().numpy()


def batch(seed, state_std, d_k=128, d_v=256, L=2, H=4):
    rng = np.random.default_rng(seed)
    parents = [synth.random_tree_parent(64, 8, 4, rng), synth.chain_parent(8), synth.random_tree_parent(33, 8, 4, rng),
               synth.chain_parent(3), synth.random_tree_parent(17, 5, 3, rng), synth.chain_parent(8)]
    if d_k == 256:
        parents = [p for p in parents if len(p) <= 32]
    return synth.make_problem(seed, L, H, d_k, d_v, parents, state_std=state_std, name=f"std{state_std}")


@pytest.mark.parametrize("route", ACCURATE)
@pytest.mark.parametrize("state_std", [0.02, 0.5, 4.0])
def test_verify_is_fp32_grade_at_any_state_scale(route, state_std):
    prob = batch(4100, state_std)
    dp = DevProblem(prob, route=route, want_u=True, max_nodes=64)
    dp.verify_tree()
    assert dp.status_value() == 0
    ref = oracle_verify(prob)
    e = rel_err(cpu(dp.o), ref)
    print(f"route {route} std {state_std}: {e:.3e} (max|x-r|/max|r| {max_err_over_max(cpu(dp.o), ref):.3e})")
    assert e <= TOL_FP32
    # u against the serial kernel (fp32), then committed through the fused entry point below
    ds = DevProblem(prob, route=speca.ROUTE_SERIAL, want_u=True, max_nodes=64)
    ds.verify_tree()
    assert rel_err(cpu(dp.u), cpu(ds.u).astype(np.float64)) <= TOL_FP32


@pytest.mark.parametrize("route", ACCURATE + [speca.ROUTE_TF32])
def test_state_that_is_exact_in_tf32(route):
    """A state whose elements carry at most 11 significant bits (bf16-initialised, say): nothing is lost by the
    tensor core's reading, so even the single-pass route must be near fp32 accuracy -- no correction constant may
    push it away."""
    prob = batch(4200, 0.5)
    bits = prob.S0.view(np.uint32) & np.uint32(0xFFFFE000)
    prob.S0 = bits.view(np.float32).copy()
    dp = DevProblem(prob, route=route, max_nodes=64)
    dp.verify_tree()
    assert dp.status_value() == 0
    e = rel_err(cpu(dp.o), oracle_verify(prob))
    print(f"route {route}: {e:.3e}")
    assert e <= (TOL if route == speca.ROUTE_TF32 else TOL_FP32)


@pytest.mark.parametrize("d_k,d_v", [(128, 128), (256, 256)])
@pytest.mark.parametrize("state_std", [0.5, 4.0])
def test_other_shapes_at_large_state(d_k, d_v, state_std):
    prob = batch(4300 + d_k, state_std, d_k=d_k, d_v=d_v, H=3)
    for route in (speca.ROUTE_FACTORIZED, speca.ROUTE_EFFECTIVE):
        dp = DevProblem(prob, route=route, max_nodes=64 if d_k == 128 else 32)
        dp.verify_tree()
        assert dp.status_value() == 0
        assert rel_err(cpu(dp.o), oracle_verify(prob)) <= TOL_FP32, route


@pytest.mark.parametrize("state_std", [0.02, 0.5, 4.0])
def test_fused_entry_point_is_fp32_grade_on_the_default_route(state_std):
    """speca_commit_verify_tree under AUTO: the committed state and the new draft's outputs at the fp32 bar."""
    rng = np.random.default_rng(4400)
    p1, p2 = batch(4401, state_std), batch(4402, state_std)
    paths = []
    for b in range(p1.B):
        lo, hi = int(p1.node_offsets[b]), int(p1.node_offsets[b + 1])
        paths.append(synth.root_path(p1.parent[lo:hi], int(rng.integers(0, hi - lo))))
    synth._set_paths(p1, paths)
    d1 = DevProblem(p1, route=speca.ROUTE_AUTO, want_u=True, max_nodes=64)
    d1.verify_tree()
    d2 = DevProblem(p2, route=speca.ROUTE_AUTO, want_u=True, max_nodes=64)
    S = d1.S.clone()
    prev = dict(k=d1.k, v=d1.v, alpha=d1.alpha, beta=d1.beta, u=d1.u, node_offsets=d1.node_offsets, total_nodes=d1.T,
                parent=d1.parent)
    speca.commit_verify_tree(d2.dims, S, prev, d1.path_idx, d1.path_len, d2.q, d2.k, d2.v, d2.alpha, d2.beta,
                             d2.node_offsets, d2.T, d2.parent, None, d2.o, d2.u, d2.ws, d2.status)
    assert d2.status_value() == 0
    S_ref = oracle_commit(p1, p1.path_idx, p1.path_len)
    o_ref = oracle.verify_tree(S_ref, p2.q, p2.k, p2.v, p2.alpha, p2.beta, p2.node_offsets, p2.parent)
    assert rel_err(cpu(S), S_ref) <= TOL_FP32 and rel_err(cpu(d2.o), o_ref) <= TOL_FP32


def test_single_pass_route_degrades_with_the_state_and_is_never_the_default():
    """Documents why ROUTE_TF32 is opt-in: its error follows the magnitude of the state."""
    prob = batch(4500, 4.0)
    fast = DevProblem(prob, route=speca.ROUTE_TF32, max_nodes=64)
    fast.verify_tree()
    auto = DevProblem(prob, route=speca.ROUTE_AUTO, max_nodes=64)
    auto.verify_tree()
    ref = oracle_verify(prob)
    e_fast, e_auto = rel_err(cpu(fast.o), ref), rel_err(cpu(auto.o), ref)
    print(f"single pass {e_fast:.3e}, default {e_auto:.3e}")
    assert e_auto <= TOL_FP32 and e_fast > 10 * e_auto
