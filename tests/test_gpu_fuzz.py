"""Randomised cross-check of the tensor-core route against the fp32 state-resident route (both on the GPU)
and, for a subset, against the oracle: many small random shapes, head counts, batch sizes, node counts on
both sides of every padding boundary, depths up to 16, both key widths, plain and fused calls."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth
from gpu_util import DevProblem, TOL, rel_err

pytestmark = pytest.mark.gpu


def cpu(t):
    return t.detach().cpu().numpy()


def random_parents(rng, B, maxn, max_depth):
    out = []
    for _ in range(B):
        n = min(maxn, int(rng.choice([0, 1, 2, 15, 16, 17, 31, 32, 33, 47, 48, 49, 63, 64, int(rng.integers(1, 65))])))
        if n == 0:
            out.append(np.zeros(0, np.int32))
        elif n == 1 or rng.random() < 0.2:
            out.append(synth.chain_parent(min(n, max_depth)))
        else:
            for _ in range(50):          # a drawn depth / fan-out may be too small for n nodes: draw again
                try:
                    out.append(synth.random_tree_parent(n, int(rng.integers(2, max_depth + 1)), int(rng.integers(2, 5)), rng))
                    break
                except ValueError:
                    continue
            else:
                out.append(synth.chain_parent(min(n, max_depth)))
    return out


def random_case(rng, deep):
    d_k = int(rng.choice([128, 256]))
    d_v = int(rng.choice([128, 256]))
    maxn = 32 if (deep or d_k == 256) else 64
    max_depth = 16 if deep else 8
    B, L, H = int(rng.integers(1, 6)), int(rng.integers(1, 3)), int(rng.integers(1, 6))
    return d_k, d_v, maxn, max_depth, L, H, B


@pytest.mark.parametrize("deep", [False, True])
def test_random_shapes_tensor_core_route_against_serial_route(deep):
    rng = np.random.default_rng(4242 + deep)
    worst = 0.0
    for case in range(40):
        d_k, d_v, maxn, max_depth, L, H, B = random_case(rng, deep)
        parents = random_parents(rng, B, maxn, max_depth)
        prob = synth.make_problem(int(rng.integers(1 << 30)), L, H, d_k, d_v, parents, max_depth=max_depth,
                                  state_std=float(rng.choice([0.02, 0.1])))
        if prob.T == 0:
            continue
        df = DevProblem(prob, route=speca.ROUTE_FACTORIZED, want_u=True, max_nodes=maxn)
        ds = DevProblem(prob, route=speca.ROUTE_SERIAL, want_u=True, max_nodes=maxn)
        df.verify_tree(); ds.verify_tree()
        assert df.status_value() == 0 and ds.status_value() == 0
        eo, eu = rel_err(cpu(df.o), cpu(ds.o)), rel_err(cpu(df.u), cpu(ds.u))
        worst = max(worst, eo, eu)
        assert eo <= TOL and eu <= TOL, (case, d_k, d_v, L, H, [len(p) for p in parents], eo, eu)
        if case % 8 == 0:
            ref = oracle.verify_tree(prob.S0, prob.q, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets, prob.parent)
            assert rel_err(cpu(df.o), ref) <= TOL
    print(f"deep={deep}: worst tensor-core vs serial difference {worst:.3e}")


def test_random_shapes_fused_against_separate_calls():
    rng = np.random.default_rng(777)
    for case in range(30):
        d_k, d_v, maxn, max_depth, L, H, B = random_case(rng, False)
        parents1, parents2 = random_parents(rng, B, maxn, max_depth), random_parents(rng, B, maxn, max_depth)
        p1 = synth.make_problem(int(rng.integers(1 << 30)), L, H, d_k, d_v, parents1)
        p2 = synth.make_problem(int(rng.integers(1 << 30)), L, H, d_k, d_v, parents2)
        if p1.T == 0 or p2.T == 0:
            continue
        paths = []
        for b in range(B):
            lo, hi = int(p1.node_offsets[b]), int(p1.node_offsets[b + 1])
            paths.append([] if hi == lo or rng.random() < 0.25 else synth.root_path(p1.parent[lo:hi], int(rng.integers(hi - lo))))
        synth._set_paths(p1, paths)
        d1 = DevProblem(p1, route=speca.ROUTE_AUTO, want_u=True, max_nodes=maxn)
        d1.verify_tree()
        d2 = DevProblem(p2, route=speca.ROUTE_AUTO, want_u=True, max_nodes=maxn)
        S = d1.S.clone()
        prev = dict(k=d1.k, v=d1.v, alpha=d1.alpha, beta=d1.beta, u=d1.u, node_offsets=d1.node_offsets, total_nodes=d1.T,
                    parent=d1.parent)
        speca.commit_verify_tree(d2.dims, S, prev, d1.path_idx, d1.path_len, d2.q, d2.k, d2.v, d2.alpha, d2.beta,
                                 d2.node_offsets, d2.T, d2.parent, None, d2.o, d2.u, d2.ws, d2.status)
        assert d1.status_value() == 0 and d2.status_value() == 0
        # the same through the two separate entry points, serial route (fp32)
        e1 = DevProblem(p1, route=speca.ROUTE_SERIAL, max_nodes=maxn)
        e1.commit()
        e2 = DevProblem(p2, route=speca.ROUTE_SERIAL, max_nodes=maxn)
        e2.S = e1.S
        e2.verify_tree()
        assert rel_err(cpu(S), cpu(e1.S)) <= TOL and rel_err(cpu(d2.o), cpu(e2.o)) <= TOL, \
            (case, d_k, d_v, L, H, [len(p) for p in parents1], [len(p) for p in parents2])
