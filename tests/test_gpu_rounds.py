"""Full-size-shaped verify -> accept -> commit loops with the state carried over many rounds,
checked on a seeded sample of (layer, sequence, head) units the oracle can follow one by one.
The oracle carries its own fp64 state for the sampled units; nothing it consumes comes from
the CUDA path (draft records are drawn on the device by torch's seeded generator, topology and
token ids on the host)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16673_b200 import binding as speca
from paper_2607_16673_b200 import synth
from gpu_util import TOL, TOL_FP32, max_err_over_max, rel_err

pytestmark = pytest.mark.gpu


def host_topology(kind, B, seed):
    rng = np.random.default_rng(seed)
    parents = (synth.mixed_chain_tree_batch(rng, B, 8, 64, 8) if kind == "cfg5"
               else synth.ragged_tree_batch(rng, B, 8, 64, 8))
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
    parent = np.concatenate(parents).astype(np.int32)
    depth = np.concatenate([synth.depth_of(p) for p in parents]).astype(np.int32)
    draft, target, root = synth.draw_tokens(rng, offs, parent, 0.75)
    return parents, offs, parent, depth, draft, target, root


def sample_problem(units, parents, offs, S_units, q, k, v, al, be, dk, dv):
    """Re-pack the sampled units as independent single-head sequences for the oracle."""
    bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    qs, ks, vs, als, bes, pars = [], [], [], [], [], []
    for (l, b, h) in units:
        s, e = int(offs[b]), int(offs[b + 1])
        qs.append(bits(q[l, s:e, h])); ks.append(bits(k[l, s:e, h])); vs.append(bits(v[l, s:e, h]))
        als.append(al[l, s:e, h].cpu().numpy()); bes.append(be[l, s:e, h].cpu().numpy())
        pars.append(parents[b])
    so = np.concatenate([[0], np.cumsum([len(p) for p in pars])]).astype(np.int32)
    cat = lambda xs: np.concatenate(xs)[None, :, None]
    return dict(S=S_units[None, :, None], q=cat(qs), k=cat(ks), v=cat(vs), alpha=cat(als), beta=cat(bes),
                offs=so, parent=np.concatenate(pars).astype(np.int32))


def run_rounds(kind, L, B, rounds, route, tol, n_sample=24, seed=77):
    H, dk, dv = 16, 128, 256
    dims = speca.Dims(L, B, H, dk, dv, 1.0, 8, 64, route)
    S = synth.device_state(seed, L, B, H, dk, dv)
    rng = np.random.default_rng(seed)
    # sample: half from the first half of the batch (chains in cfg5), half from the second (trees)
    units = [(int(rng.integers(L)), int(rng.integers(B // 2) + (B // 2) * (i % 2)), int(rng.integers(H)))
             for i in range(n_sample)]
    units = sorted(set(units))
    S_ref = np.stack([S[l, b, h].cpu().numpy().astype(np.float64) for (l, b, h) in units])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    path_idx = torch.zeros(B, 8, dtype=torch.int32, device="cuda")
    path_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    next_tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    worst_o = worst_s = mom_o = mom_s = 0.0
    accepted = []
    for r in range(rounds):
        parents, offs, parent, depth, draft, target, root = host_topology(kind, B, seed + 100 + r)
        T = int(offs[-1])
        q, k, v, al, be = synth.device_records(seed + 200 + r, L, T, H, dk, dv)
        t = lambda a: torch.from_numpy(a).cuda()
        d_offs, d_par, d_depth = t(offs), t(parent), t(depth)
        o = torch.full((L, T, H, dv), float("nan"), device="cuda")
        ws = speca.alloc_workspace(dims, T)
        S_before = S.clone() if r == 0 else None
        speca.verify_tree(dims, S, q, k, v, al, be, d_offs, T, d_par, d_depth, o, None, ws, status)
        speca.greedy_accept(B, 8, d_offs, d_par, t(draft), t(target), t(root), path_idx, path_len, next_tok, status)
        if S_before is not None:
            assert torch.equal(S, S_before)
        # oracle on the sample, from its own state
        sp = sample_problem(units, parents, offs, S_ref, q, k, v, al, be, dk, dv)
        o_ref = oracle.verify_tree(sp["S"], sp["q"], sp["k"], sp["v"], sp["alpha"], sp["beta"], sp["offs"], sp["parent"])
        pi, pl, nt = oracle.greedy_accept(offs, parent, draft, target, root, 8)
        assert np.array_equal(path_idx.cpu().numpy(), pi) and np.array_equal(path_len.cpu().numpy(), pl)
        assert np.array_equal(next_tok.cpu().numpy(), nt)
        o_gpu = np.concatenate([o[l, int(offs[b]):int(offs[b + 1]), h].cpu().numpy() for (l, b, h) in units])
        assert not np.isnan(o_gpu).any()
        worst_o = max(worst_o, rel_err(o_gpu, o_ref[0, :, 0]))
        mom_o = max(mom_o, max_err_over_max(o_gpu, o_ref[0, :, 0]))
        speca.commit(dims, S, k, v, al, be, d_offs, T, d_par, path_idx, path_len, status)
        sub_pi = np.stack([pi[b] for (_, b, _) in units]); sub_pl = np.asarray([pl[b] for (_, b, _) in units], np.int32)
        S_ref = oracle.commit(sp["S"], sp["k"], sp["v"], sp["alpha"], sp["beta"], sp["offs"], sub_pi, sub_pl)[0, :, 0]
        S_gpu = np.stack([S[l, b, h].cpu().numpy() for (l, b, h) in units])
        worst_s = max(worst_s, rel_err(S_gpu, S_ref))
        mom_s = max(mom_s, max_err_over_max(S_gpu, S_ref))
        accepted.append(float(pl.mean()))
        assert int(status.item()) == 0
    print(f"{kind} route={route} rounds={rounds}: worst verify err {worst_o:.3e} (max|x-r|/max|r| {mom_o:.3e}), "
          f"worst state err {worst_s:.3e} (max|x-r|/max|r| {mom_s:.3e}), mean accepted {np.mean(accepted):.2f}")
    assert worst_o <= tol and worst_s <= TOL_FP32 * 4
    return worst_o, worst_s


@pytest.mark.parametrize("route,tol", [(speca.ROUTE_SERIAL, TOL_FP32 * 4), (speca.ROUTE_AUTO, TOL_FP32 * 4), (speca.ROUTE_TF32, TOL)])
def test_cfg5_shaped_16_rounds(route, tol):
    run_rounds("cfg5", 2, 128, 16, route, tol)


@pytest.mark.parametrize("route,tol", [(speca.ROUTE_SERIAL, TOL_FP32 * 4), (speca.ROUTE_AUTO, TOL_FP32 * 4), (speca.ROUTE_TF32, TOL)])
def test_cfg4_shaped_rounds(route, tol):
    run_rounds("cfg4", 3, 32, 4, route, tol)


def test_cfg5_shaped_64_rounds_default_route():
    """Long serving loop on the default route: verify errors do not grow with the carried state."""
    wo, ws = run_rounds("cfg5", 1, 128, 64, speca.ROUTE_AUTO, TOL_FP32 * 4, n_sample=16)
    assert ws <= 1e-4


def test_cfg5_full_size_sampled():
    """The benchmark's own launch configuration (24 layers x 128 sequences x 16 heads, 6.4 GB of state),
    two rounds, checked on sampled units."""
    run_rounds("cfg5", 24, 128, 2, speca.ROUTE_AUTO, TOL_FP32 * 4, n_sample=32, seed=91)


def test_cfg4_full_size_sampled():
    run_rounds("cfg4", 24, 32, 2, speca.ROUTE_AUTO, TOL_FP32 * 4, n_sample=32, seed=92)


def run_rounds_fused(kind, L, B, rounds, tol, n_sample=24, seed=177, H=16, dk=128, dv=256, max_nodes=64,
                     route=speca.ROUTE_TF32):
    """The same loop through speca_commit_verify_tree: the commit of round r - 1 runs inside the
    verification of round r; the last pending commit is flushed with speca_commit."""
    dims = speca.Dims(L, B, H, dk, dv, 1.0, 8, max_nodes, route)
    S = synth.device_state(seed, L, B, H, dk, dv)
    rng = np.random.default_rng(seed)
    units = sorted({(int(rng.integers(L)), int(rng.integers(B // 2) + (B // 2) * (i % 2)), int(rng.integers(H)))
                    for i in range(n_sample)})
    S_ref = np.stack([S[l, b, h].cpu().numpy().astype(np.float64) for (l, b, h) in units])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    paths = [(torch.zeros(B, 8, dtype=torch.int32, device="cuda"), torch.zeros(B, dtype=torch.int32, device="cuda"))
             for _ in range(2)]
    next_tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = lambda a: torch.from_numpy(a).cuda()
    worst_o = worst_s = mom_o = mom_s = 0.0
    prev = prev_host = None
    for r in range(rounds + 1):
        flush = r == rounds
        if not flush:
            if kind == "paper256":
                trng = np.random.default_rng(seed + 100 + r)
                parents = [synth.chain_parent(8) for _ in range(B // 2)]
                parents += [synth.proposal_tree_parent(4, int(trng.integers(4, 9)), int(trng.integers(16, 33)), trng, 8)
                            for _ in range(B - B // 2)]
                offs = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int32)
                parent = np.concatenate(parents).astype(np.int32)
                draft, target, root = synth.draw_tokens(trng, offs, parent, 0.75)
            else:
                parents, offs, parent, _, draft, target, root = host_topology(kind, B, seed + 100 + r)
            T = int(offs[-1])
            q, k, v, al, be = synth.device_records(seed + 200 + r, L, T, H, dk, dv)
            d_offs, d_par = t(offs), t(parent)
            o = torch.full((L, T, H, dv), float("nan"), device="cuda")
            u = torch.empty(L, T, H, dv, device="cuda")
            ws = speca.alloc_workspace(dims, T)
        pi_d, pl_d = paths[r & 1]
        ppi, ppl = paths[(r - 1) & 1]
        # the oracle commits the previous round's paths to its own state first
        if prev_host is not None:
            sp0, sub_pi, sub_pl = prev_host
            S_ref = oracle.commit(S_ref[None, :, None], sp0["k"], sp0["v"], sp0["alpha"], sp0["beta"], sp0["offs"],
                                  sub_pi, sub_pl)[0, :, 0]
        if flush:
            pp = prev
            speca.commit(dims, S, pp["k"], pp["v"], pp["alpha"], pp["beta"], pp["node_offsets"], pp["total_nodes"],
                         pp["parent"], ppi, ppl, status)
        else:
            speca.commit_verify_tree(dims, S, prev, ppi, ppl, q, k, v, al, be, d_offs, T, d_par, None, o, u, ws, status)
            speca.greedy_accept(B, 8, d_offs, d_par, t(draft), t(target), t(root), pi_d, pl_d, next_tok, status)
        assert int(status.item()) == 0
        S_gpu = np.stack([S[l, b, h].cpu().numpy() for (l, b, h) in units])
        worst_s = max(worst_s, rel_err(S_gpu, S_ref))
        mom_s = max(mom_s, max_err_over_max(S_gpu, S_ref))
        if flush:
            break
        sp = sample_problem(units, parents, offs, S_ref, q, k, v, al, be, dk, dv)
        o_ref = oracle.verify_tree(sp["S"], sp["q"], sp["k"], sp["v"], sp["alpha"], sp["beta"], sp["offs"], sp["parent"])
        pi, pl, _ = oracle.greedy_accept(offs, parent, draft, target, root, 8)
        assert np.array_equal(pi_d.cpu().numpy(), pi) and np.array_equal(pl_d.cpu().numpy(), pl)
        o_gpu = np.concatenate([o[l, int(offs[b]):int(offs[b + 1]), h].cpu().numpy() for (l, b, h) in units])
        assert not np.isnan(o_gpu).any()
        worst_o = max(worst_o, rel_err(o_gpu, o_ref[0, :, 0]))
        mom_o = max(mom_o, max_err_over_max(o_gpu, o_ref[0, :, 0]))
        prev = dict(k=k, v=v, alpha=al, beta=be, u=u, node_offsets=d_offs, total_nodes=T, parent=d_par)
        prev_host = (sp, np.stack([pi[b] for (_, b, _) in units]), np.asarray([pl[b] for (_, b, _) in units], np.int32))
    print(f"fused {kind} L={L} B={B} rounds={rounds}: worst verify err {worst_o:.3e} (max|x-r|/max|r| {mom_o:.3e}), "
          f"worst state err {worst_s:.3e} (max|x-r|/max|r| {mom_s:.3e})")
    assert worst_o <= tol and worst_s <= tol
    return worst_o, worst_s


def test_fused_cfg5_shaped_16_rounds():
    run_rounds_fused("cfg5", 2, 128, 16, TOL)


def test_fused_entry_point_on_the_default_route_64_rounds():
    """speca_commit_verify_tree under AUTO (commit kernel, then fp32-grade verification): 64 carried rounds at the
    shape of the largest configuration; the committed state stays within fp32 rounding of the oracle's."""
    wo, ws = run_rounds_fused("cfg5", 1, 128, 64, TOL_FP32 * 4, n_sample=16, route=speca.ROUTE_AUTO)
    assert ws <= 1e-4


def test_fused_paper256_shaped_rounds():
    run_rounds_fused("paper256", 2, 64, 8, TOL, H=8, dk=256, dv=256, max_nodes=32)


def test_fused_cfg5_full_size_sampled():
    """The fused rounds in the benchmark's own launch configuration (6.4 GB of state), three rounds."""
    run_rounds_fused("cfg5", 24, 128, 3, TOL, n_sample=32, seed=191)
