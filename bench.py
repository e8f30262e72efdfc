#!/usr/bin/env python
"""Benchmark of the speculative verify -> accept -> commit path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5|cfg4|cfg3|cfg2|paper256|trees64|chains8|paper]
                    [--sweep commit-len|unit-types] [--impl reference]

One "step" is one round of the whole hot path over one batch of synthetic draft input:
plan + verify (all layers, heads, nodes) -> greedy accept -> commit, with the committed
state carried from step to step.  The default workload is the largest single-GPU
configuration: 128 sequences, 24 layers, 16 heads, d_k = 128, d_v = 256, half of the
sequences with 8-token chains and half with 64-node trees.

The metric is verified draft token-layers per second (tokens verified in one step times
the layer count, divided by the step time).  Rank 0 prints ONE JSON line.  For N > 1 the
sequences are partitioned over the ranks (every rank owns whole sequences; there is no
exchange step anywhere on the path), launched one process per GPU by torchrun.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verified draft token-layers/s (verify+accept+commit)"
UNIT = "token-layers/s"

WORKLOADS = {
    # name: (L, B, H, d_k, d_v, description)
    "cfg5": (24, 128, 16, 128, 256, "128 seq x 24 layers x 16 heads, d_k=128 d_v=256; 64 seq with 8-token chains + "
                                    "64 seq with 64-node trees (depth<=8)"),
    "cfg4": (24, 32, 16, 128, 256, "32 seq x 24 layers x 16 heads, d_k=128 d_v=256; ragged trees of 8..64 nodes (depth<=8)"),
    # the paper's target shape (h_v = 8, d_k = d_v = 256, 24 layers) served in a batch
    # the two unit types of cfg5 on their own (same shape): what a unit of each kind costs
    "trees64": (24, 128, 16, 128, 256, "128 seq x 24 layers x 16 heads, d_k=128 d_v=256; every sequence a 64-node tree (depth<=8)"),
    "chains8": (24, 128, 16, 128, 256, "128 seq x 24 layers x 16 heads, d_k=128 d_v=256; every sequence an 8-token chain"),
    "paper256": (24, 64, 8, 256, 256, "64 seq x 24 layers x 8 heads, d_k=d_v=256 (the paper's target shape); 32 seq with "
                                      "8-token chains + 32 seq with top-4 proposal trees of 16..32 nodes (depth 4..8)"),
}
POOL = 3            # independent draft inputs rotated over the steps ("fresh draft factors each round")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=48)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg5", choices=sorted(WORKLOADS) + ["paper", "cfg2", "cfg3"],
                    help="cfg5 (default), cfg4, paper256, trees64 / chains8 (cfg5's unit types on their own), or 'paper': "
                         "the paper's own target shape and proposal shapes (Table 1)")
    ap.add_argument("--impl", default="speca", choices=["speca", "reference"])
    ap.add_argument("--route", type=int, default=0,
                    help="0 auto (fp32-grade), 1 serial, 2 factorised (fp32-grade), 3 single-pass TF32, 4 effective-query")
    ap.add_argument("--sweep", default=None, choices=["commit-len", "unit-types", "role-waits"],
                    help="commit-len: commit throughput against the accepted path length; unit-types: time per "
                         "(layer, sequence, head) unit and SM of 8-token chains and 64-node trees, per route")
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-fused", action="store_true", help="skip the fused commit-and-verify leg")
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (profiling only)")
    ap.add_argument("--batch", type=int, default=None, help="override the batch (profiling only)")
    return ap.parse_args()


# ---------------------------------------------------------------------------
# workload description (host side: topology and token ids; no method arithmetic)
# ---------------------------------------------------------------------------
def workload_parents(name: str, rng, n: int):
    """Parent arrays of n sequences of a workload."""
    from paper_2607_16673_b200 import synth
    if name == "cfg5":
        return synth.mixed_chain_tree_batch(rng, n, 8, 64, 8)
    if name == "trees64":
        return [synth.random_tree_parent(64, 8, 4, rng) for _ in range(n)]
    if name == "chains8":
        return [synth.chain_parent(8) for _ in range(n)]
    if name == "paper256":
        return ([synth.chain_parent(8) for _ in range(n // 2)] +
                [synth.proposal_tree_parent(4, int(rng.integers(4, 9)), int(rng.integers(16, 33)), rng, 8)
                 for _ in range(n - n // 2)])
    return synth.ragged_tree_batch(rng, n, 8, 64, 8)


def host_round_inputs(name: str, B: int, seed: int):
    """Topology and token ids of one round, on the host."""
    from paper_2607_16673_b200 import synth
    rng = np.random.default_rng(seed)
    parents = workload_parents(name, rng, B)
    sizes = [len(p) for p in parents]
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    parent = np.concatenate(parents).astype(np.int32)
    depth = np.concatenate([synth.depth_of(p) for p in parents]).astype(np.int32)
    draft, target, root_target = synth.draw_tokens(rng, offs, parent, 0.75)
    return dict(parents=parents, node_offsets=offs, parent=parent, depth=depth, draft_tok=draft,
                target_tok=target, root_target_tok=root_target, T=int(offs[-1]))


def algorithmic_bytes(L, B, H, dk, dv, T, path_len):
    """Bytes the method itself must move in one step (HBM roofline numerator)."""
    units = L * B * H
    Sb = 4 * dk * dv
    rec_in = 4 * dk + 2 * dv + 8             # q, k bf16 + v bf16 + alpha, beta fp32 per node per (layer, head)
    verify = units * Sb + T * L * H * rec_in + T * L * H * 4 * dv
    n_commit_seq = int(np.count_nonzero(path_len))
    commit = 2 * n_commit_seq * L * H * Sb + int(path_len.sum()) * L * H * (2 * dk + 2 * dv + 8)
    return verify, commit


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def rank_seed(base: int, rank: int, j: int = 0) -> int:
    """Seed of input set j on a rank: every rank draws its own sequences (the batch is partitioned
    over the ranks, a rank owns whole sequences), so seeds must differ across (rank, j)."""
    return base + 97 * rank + j


def reduce_over_ranks(dist, device, total_ms, t_verify, t_commit, tokens, vb, cb):
    """Whole-job numbers: times are the MAX over ranks, processed units and bytes the SUM.
    `dist` is torch.distributed (initialised) or None for a single process."""
    if dist is None:
        return total_ms, t_verify, t_commit, float(tokens), float(vb), float(cb)
    import torch
    tt = torch.tensor([total_ms, t_verify, t_commit], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    cnt = torch.tensor([tokens, vb, cb], device=device, dtype=torch.float64)
    dist.all_reduce(cnt, op=dist.ReduceOp.SUM)
    return (float(tt[0]), float(tt[1]), float(tt[2]), float(cnt[0]), float(cnt[1]), float(cnt[2]))


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the benchmark runs.  It is
    started before the warm-up (nvidia-smi needs a moment to come up); `mark()` brackets the timed
    region and only samples inside the marks are summarised (all samples if none fell inside)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.marks = []
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=self.tmp, stderr=subprocess.DEVNULL)
            time.sleep(0.5)
        except Exception:
            self.proc = None

    def mark(self):
        self.marks.append(time.time())

    @staticmethod
    def _ts(text: str):
        import datetime
        try:
            return datetime.datetime.strptime(text.strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        for line in self.tmp.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                rows.append((self._ts(parts[0]), float(parts[1]), float(parts[2]),
                             [nm for nm, val in zip(names, parts[4:8]) if val.lower().startswith("active")]))
            except ValueError:
                continue
        self.tmp.close()
        os.unlink(self.tmp.name)
        inside = rows
        if len(self.marks) >= 2:
            lo, hi = self.marks[0] - 0.02, self.marks[-1] + 0.02
            sel = [r for r in rows if r[0] is not None and lo <= r[0] <= hi]
            if sel:
                inside = sel
                out["window"] = "timed region"
            else:
                out["window"] = "whole run (no sample fell inside the timed region)"
        if inside:
            out.update(sm_mhz=float(np.median([r[1] for r in inside])), sm_max_mhz=float(max(r[2] for r in inside)),
                       samples=len(inside))
            out["reasons"] = sorted({nm for r in inside for nm in r[3]})
        return out


# ---------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------
def run_speca(args):
    import torch
    import torch.distributed as dist

    from paper_2607_16673_b200 import binding as speca
    from paper_2607_16673_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)

    L, B, H, dk, dv, desc = WORKLOADS[args.workload]
    L = args.layers or L
    B = args.batch or B
    dims = speca.Dims(L, B, H, dk, dv, 1.0, 8, 64 if dk <= 128 else 32, args.route)
    stream = torch.cuda.current_stream()

    # --- inputs resident in HBM -------------------------------------------------
    S = synth.device_state(rank_seed(1000, rank), L, B, H, dk, dv, 0.02, dev)
    pool = []
    for j in range(POOL):
        hi = host_round_inputs(args.workload, B, rank_seed(5000, rank, j))
        q, k, v, al, be = synth.device_records(rank_seed(7000, rank, j), L, hi["T"], H, dk, dv, dev)
        t = lambda a: torch.from_numpy(a).to(dev)
        pool.append(dict(hi, q=q, k=k, v=v, alpha=al, beta=be, d_offs=t(hi["node_offsets"]),
                         d_parent=t(hi["parent"]), d_depth=t(hi["depth"]), d_draft=t(hi["draft_tok"]),
                         d_target=t(hi["target_tok"]), d_root=t(hi["root_target_tok"])))
    Tmax = max(p["T"] for p in pool)
    o_buf = torch.empty(L * Tmax * H * dv, dtype=torch.float32, device=dev)
    ws = speca.alloc_workspace(dims, Tmax, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    path_idx = torch.zeros(B, 8, dtype=torch.int32, device=dev)
    path_len = torch.zeros(B, dtype=torch.int32, device=dev)
    next_tok = torch.zeros(B, dtype=torch.int32, device=dev)

    def o_view(T):
        return o_buf[: L * T * H * dv].view(L, T, H, dv)

    def step(p, ev=None):
        T = p["T"]
        if ev: ev[0].record(stream)
        speca.verify_tree(dims, S, p["q"], p["k"], p["v"], p["alpha"], p["beta"], p["d_offs"], T, p["d_parent"],
                          p["d_depth"], o_view(T), None, ws, status)
        if ev: ev[1].record(stream)
        speca.greedy_accept(B, 8, p["d_offs"], p["d_parent"], p["d_draft"], p["d_target"], p["d_root"],
                            path_idx, path_len, next_tok, status)
        if ev: ev[2].record(stream)
        speca.commit(dims, S, p["k"], p["v"], p["alpha"], p["beta"], p["d_offs"], T, p["d_parent"], path_idx,
                     path_len, status)
        if ev: ev[3].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # accepted lengths per pool entry (integer-only, independent of the state): for the byte counts
    for p in pool:
        speca.greedy_accept(B, 8, p["d_offs"], p["d_parent"], p["d_draft"], p["d_target"], p["d_root"],
                            path_idx, path_len, next_tok, status)
        torch.cuda.synchronize()
        p["path_len"] = path_len.cpu().numpy().copy()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    for w in range(args.warmup):
        step(pool[w % POOL])
    barrier()

    K = args.steps
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    barrier()
    if sampler: sampler.mark()
    t_start.record(stream)
    for i in range(K):
        step(pool[(args.warmup + i) % POOL], evs[i])
    t_end.record(stream)
    barrier()
    if sampler: sampler.mark()
    clocks = sampler.stop() if sampler else None
    total_ms = t_start.elapsed_time(t_end)
    assert int(status.item()) == 0, f"device status word {int(status.item())}"

    tokens = sum(pool[(args.warmup + i) % POOL]["T"] for i in range(K))
    vb = cb = 0
    for i in range(K):
        p = pool[(args.warmup + i) % POOL]
        a, c = algorithmic_bytes(L, B, H, dk, dv, p["T"], p["path_len"])
        vb += a; cb += c
    t_verify = sum(e[0].elapsed_time(e[1]) for e in evs) / K       # plan + verify kernels
    t_accept = sum(e[1].elapsed_time(e[2]) for e in evs) / K
    t_commit = sum(e[2].elapsed_time(e[3]) for e in evs) / K

    total_ms, t_verify, t_commit, tokens_all, vb_all, cb_all = reduce_over_ranks(
        dist if world > 1 else None, dev, total_ms, t_verify, t_commit, tokens, vb, cb)

    # --- decode-step baseline at the same batch (context) --------------------------
    q1, k1, v1, a1, b1 = synth.device_records(99, L, B, H, dk, dv, dev)
    o1 = torch.empty(L, B, H, dv, device=dev)
    d1 = speca.Dims(L, B, H, dk, dv)
    S_dec = S.clone() if S.numel() * 4 < 20e9 else S
    for _ in range(2):
        speca.decode_step(d1, S_dec, q1, k1, v1, a1, b1, o1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    n_dec = 5
    for _ in range(n_dec):
        speca.decode_step(d1, S_dec, q1, k1, v1, a1, b1, o1)
    e1.record(stream)
    torch.cuda.synchronize()
    dec_ms = e0.elapsed_time(e1) / n_dec
    dec_bytes = L * B * H * (2 * 4 * dk * dv + 4 * dk + 2 * dv + 8 + 4 * dv)
    del S_dec

    # --- the same verification on the single-pass TF32 route (context: opt-in, 2e-3-grade) ---------
    dims_tf32 = speca.Dims(L, B, H, dk, dv, 1.0, 8, 64 if dk <= 128 else 32, speca.ROUTE_TF32)
    p0 = pool[0]
    for _ in range(2):
        speca.verify_tree(dims_tf32, S, p0["q"], p0["k"], p0["v"], p0["alpha"], p0["beta"], p0["d_offs"], p0["T"],
                          p0["d_parent"], p0["d_depth"], o_view(p0["T"]), None, ws, status)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(5):
        speca.verify_tree(dims_tf32, S, p0["q"], p0["k"], p0["v"], p0["alpha"], p0["beta"], p0["d_offs"], p0["T"],
                          p0["d_parent"], p0["d_depth"], o_view(p0["T"]), None, ws, status)
    e1.record(stream)
    torch.cuda.synchronize()
    tf32_ms = e0.elapsed_time(e1) / 5

    # --- convolution-state commit (the other half of the state holder), same accepted paths --------
    ch, W = H * (2 * dk + dv), 3
    C = torch.zeros(L, B, W, ch, dtype=torch.bfloat16, device=dev)
    x_conv = torch.zeros(L, p0["T"], ch, dtype=torch.bfloat16, device=dev)
    speca.greedy_accept(B, 8, p0["d_offs"], p0["d_parent"], p0["d_draft"], p0["d_target"], p0["d_root"],
                        path_idx, path_len, next_tok, status)
    for _ in range(3):
        speca.commit_conv(C, x_conv, p0["d_offs"], p0["T"], path_idx, path_len, status)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(10):
        speca.commit_conv(C, x_conv, p0["d_offs"], p0["T"], path_idx, path_len, status)
    e1.record(stream)
    torch.cuda.synchronize()
    conv_ms = e0.elapsed_time(e1) / 10
    pl0 = p0["path_len"]
    conv_bytes = L * ch * 2 * int(np.sum(np.where(pl0 > 0, W + np.maximum(W - pl0, 0) + np.minimum(pl0, W), 0)))
    del C, x_conv

    # --- draft-side utilities on the same topology (context: they run once per round, before verification) ----
    rng_u = np.random.default_rng(rank_seed(9000, rank))
    logp = torch.from_numpy(np.log(rng_u.uniform(0.02, 1.0, p0["T"])).astype(np.float32)).to(dev)
    mask_h = np.zeros((B, 64, 64), np.uint8)
    for b_, par_ in enumerate(p0["parents"]):
        for i_ in range(len(par_)):
            a_ = i_
            while a_ >= 0:
                mask_h[b_, i_, a_] = 1
                a_ = int(par_[a_])
    mask_d = torch.from_numpy(mask_h).to(dev)
    par_out = torch.empty(p0["T"], dtype=torch.int32, device=dev)
    oo, op, oi = (torch.empty(B + 1, dtype=torch.int32, device=dev), torch.empty(p0["T"], dtype=torch.int32, device=dev),
                  torch.empty(p0["T"], dtype=torch.int32, device=dev))

    def time_util(fn, reps=10):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    mask_ms = time_util(lambda: speca.tree_mask_to_parent(mask_d, p0["d_offs"], par_out, status))
    prune_ms = time_util(lambda: speca.prune_tree(64, 2.0, 32, p0["d_offs"], p0["d_parent"], logp, oo, op, oi, status))
    g_sa = torch.Generator(device=dev).manual_seed(1234)
    sa_q = torch.rand(p0["T"], device=dev, generator=g_sa) * 0.9 + 0.1
    sa_p = sa_q * (0.5 + torch.rand(p0["T"], device=dev, generator=g_sa))
    sa_u = torch.rand(p0["T"], device=dev, generator=g_sa)
    sa_idx = torch.empty(B, 8, dtype=torch.int32, device=dev)
    sa_len = torch.empty(B, dtype=torch.int32, device=dev)
    sacc_ms = time_util(lambda: speca.stochastic_accept(B, 8, p0["d_offs"], p0["d_parent"], sa_p, sa_q, sa_u,
                                                        sa_idx, sa_len, status))
    ch_head = torch.empty(p0["T"], dtype=torch.int32, device=dev)
    ch_cnt = torch.empty(B, dtype=torch.int32, device=dev)
    chain_ms = time_util(lambda: speca.chain_decompose(64, p0["d_offs"], p0["d_parent"], ch_head, ch_cnt, status))
    assert torch.equal(par_out, p0["d_parent"]), "mask converter does not reproduce the parent array"

    # --- the same rounds with the commit delayed into the next round's verification ----
    fused = None
    if not args.no_fused:
        fused = run_fused(args, speca, dims, S, pool, o_buf, ws, status, stream, barrier, dist if world > 1 else None, dev)

    # --- end to end with host buffers (C ABI fed from pinned host memory) ---------
    e2e = None
    if not args.no_e2e and rank == 0:
        e2e = run_e2e(args, speca, dims, S, pool, o_buf, ws, status, path_idx, path_len, next_tok, stream)
    if world > 1:
        dist.barrier()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peak_gbs()
    ms_per_step = total_ms / K
    value = tokens_all * L / (total_ms * 1e-3)
    dom = "verify" if t_verify >= t_commit else "commit"
    dom_ms = max(t_verify, t_commit)
    dom_bytes = (vb if dom == "verify" else cb) / K
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {desc}", "n_layers": L, "batch_per_gpu": B, "heads": H,
                   "d_k": dk, "d_v": dv, "nodes_per_step_per_gpu": [p["T"] for p in pool],
                   "mean_accepted_len": float(np.mean([p["path_len"].mean() for p in pool])),
                   "input_pool": POOL, "l2": f"inputs larger than L2 (state {L * B * H * dk * dv * 4 / 1e9:.1f} GB)",
                   "route": {0: "auto: tensor-core route with split operands (fp32-grade)", 1: "serial", 2: "factorised, split operands",
                             3: "single-pass TF32", 4: "effective-query"}.get(args.route, str(args.route)),
                   "parallelism": f"dp{world} (sequences partitioned, no collective)"},
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": (ncu_traffic(args.workload + {3: "-tf32", 4: "-effective"}.get(args.route, "") if dom == "verify" else args.workload, dom)
                                 if not args.layers and not args.batch else None),
                     "algorithmic_bytes_per_launch": dom_bytes, "ms_per_launch": dom_ms},
        "kernels": {"verify_ms": t_verify, "accept_ms": t_accept, "commit_ms": t_commit,
                    "verify_single_pass_tf32_ms": tf32_ms,
                    "verify_gbs": vb / K / (t_verify * 1e-3) / 1e9, "commit_gbs": cb / K / (t_commit * 1e-3) / 1e9,
                    "step_gbs": (vb + cb) / K / (ms_per_step * 1e-3) / 1e9,
                    "step_frac_of_peak": (vb + cb) / K / (ms_per_step * 1e-3) / 1e9 / peak,
                    "step_frac_of_8TBs": (vb + cb) / K / (ms_per_step * 1e-3) / 1e9 / 8000.0},
        "decode_step": {"ms": dec_ms, "gbs": dec_bytes / (dec_ms * 1e-3) / 1e9,
                        "token_layers_per_s": B * L / (dec_ms * 1e-3),
                        "note": "one autoregressive token per sequence at the same batch"},
        # plan, verify, accept, commit -- and the long-path commit kernel in front of it where the batch is large enough
        # for the library to use it (d_k <= 128, at least 128 16-row tiles per resident warp; 16 warps per SM)
        "gpu_launches": (5 if dk <= 128 and L * B * H * (dv // 16) >= 128 * 16 * torch.cuda.get_device_properties(dev).multi_processor_count else 4) * K,
        "conv_commit": {"ms": conv_ms, "channels": ch, "width": W, "gbs": conv_bytes / (conv_ms * 1e-3) / 1e9,
                        "note": "speca_commit_conv on the accepted paths of one round; outside the timed step"},
        "draft_utils": {"tree_mask_to_parent_ms": mask_ms, "prune_tree_ms": prune_ms, "stochastic_accept_ms": sacc_ms, "chain_decompose_ms": chain_ms,
                        "note": "one call over the batch's topology (tau = 2, budget 32); integer work outside the timed step"},
        "fused": fused,
        "clocks": clocks,
        "e2e": e2e,
    }
    if not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(args.workload, L, H, dk, dv)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_fused(args, speca, dims, S, pool, o_buf, ws, status, stream, barrier, dist, dev):
    """The same rounds through speca_commit_verify_tree: round r verifies its draft from the state
    with round r-1's accepted paths applied on chip (the state is read once and written once per
    round), then runs greedy acceptance.  Reported beside the headline, not instead of it."""
    import torch
    L, B, H, dk, dv = dims.n_layers, dims.batch, dims.heads, dims.d_k, dims.d_v
    # the one-pass kernel exists on the single-pass TF32 route only (on the default route the entry point runs
    # the commit kernel and then the fp32-grade verification, i.e. the separate step)
    dims = speca.Dims(L, B, H, dk, dv, 1.0, dims.max_depth, dims.max_nodes, speca.ROUTE_TF32)
    Tmax = max(p["T"] for p in pool)
    u_buf = [torch.empty(L * Tmax * H * dv, dtype=torch.float32, device=dev) for _ in range(2)]
    paths = [(torch.zeros(B, 8, dtype=torch.int32, device=dev), torch.zeros(B, dtype=torch.int32, device=dev))
             for _ in range(2)]
    next_tok = torch.zeros(B, dtype=torch.int32, device=dev)
    view = lambda buf, T: buf[: L * T * H * dv].view(L, T, H, dv)

    def step(i):
        p = pool[i % POOL]
        T = p["T"]
        pi, pl = paths[i & 1]
        prev, (ppi, ppl) = None, paths[(i - 1) & 1]
        if i > 0:
            pp = pool[(i - 1) % POOL]
            prev = dict(k=pp["k"], v=pp["v"], alpha=pp["alpha"], beta=pp["beta"], u=view(u_buf[(i - 1) & 1], pp["T"]),
                        node_offsets=pp["d_offs"], total_nodes=pp["T"], parent=pp["d_parent"])
        speca.commit_verify_tree(dims, S, prev, ppi, ppl, p["q"], p["k"], p["v"], p["alpha"], p["beta"], p["d_offs"], T,
                                 p["d_parent"], p["d_depth"], view(o_buf, T), view(u_buf[i & 1], T), ws, status)
        speca.greedy_accept(B, 8, p["d_offs"], p["d_parent"], p["d_draft"], p["d_target"], p["d_root"], pi, pl,
                            next_tok, status)

    W, K = max(3, args.warmup), args.steps
    for i in range(W):
        step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(W, W + K):
        step(i)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    assert int(status.item()) == 0, f"device status word {int(status.item())}"
    tokens = sum(pool[i % POOL]["T"] for i in range(W, W + K))
    # bytes: state read once, written once where something is committed, records in, o out, keys and gates of the
    # accepted nodes -- and the u rows, which every round writes for all nodes and re-reads for the accepted ones
    Sb = 4 * dk * dv
    nbytes = 0
    for i in range(W, W + K):
        p, pp = pool[i % POOL], pool[(i - 1) % POOL]
        nbytes += L * B * H * Sb + int(np.count_nonzero(pp["path_len"])) * L * H * Sb
        nbytes += p["T"] * L * H * (4 * dk + 2 * dv + 8 + 4 * dv) + int(pp["path_len"].sum()) * L * H * (2 * dk + 2 * dv + 8)
        nbytes += p["T"] * L * H * 4 * dv + int(pp["path_len"].sum()) * L * H * 4 * dv
    if dist is not None:
        tt = torch.tensor([ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        cnt = torch.tensor([tokens, nbytes], device=dev, dtype=torch.float64)
        dist.all_reduce(cnt, op=dist.ReduceOp.SUM)
        ms, tokens, nbytes = float(tt[0]), float(cnt[0]), float(cnt[1])
    peak, peak_kind = measured_peak_gbs()
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"value": tokens * L / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / K, "steps": K, "gpu_launches": 4 * K,
            "algorithmic_gbs": gbs, "frac_of_peak": gbs / peak, "peak_kind": f"of {peak_kind}",
            "route": "single-pass TF32 (SPECA_ROUTE_TF32): outputs within the 2e-3 bar, not fp32-grade",
            "note": "speca_commit_verify_tree + speca_greedy_accept per round; the commit of round r runs inside the "
                    "verification of round r+1 (state read once and written once per round); the u rows written and "
                    "re-read are counted in algorithmic_gbs"}


def ncu_traffic(workload: str, kernel: str):
    """DRAM bytes per full-size launch (dram__bytes_read.sum + dram__bytes_write.sum) of a kernel, from the ncu
    captures summarised in profiles/dram_traffic.md: rows `| workload | kernel | captured bytes | scale | ... |`,
    the capture being a reduced-layer case scaled to the full launch by the number of units.  None if absent."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    try:
        with open(path) as f:
            for line in f:
                cells = [c.strip() for c in line.strip().strip("|").split("|")]
                if len(cells) >= 4 and cells[0] == workload and cells[1] == kernel:
                    try:
                        return float(cells[2]) * float(cells[3])
                    except ValueError:
                        continue
    except OSError:
        pass
    return None


def run_e2e(args, speca, dims, S, pool, o_buf, ws, status, path_idx, path_len, next_tok, stream):
    """Same step, but every step's draft inputs start in pinned HOST memory and its results
    (outputs o, accepted paths, next tokens) are read back to the host inside the timed region.
    The committed state is the durable device-resident object and stays in HBM.  As a serving loop
    would, the copies run on their own streams with two sets of device buffers, so that the upload
    of step i+1, the kernels of step i and the read-back of step i-1 overlap (PCIe is full duplex)."""
    import torch
    L, B, H, dk, dv = dims.n_layers, dims.batch, dims.heads, dims.d_k, dims.d_v
    p0 = pool[0]
    T = p0["T"]
    dev = S.device
    names = ["q", "k", "v", "alpha", "beta", "d_offs", "d_parent", "d_depth", "d_draft", "d_target", "d_root"]
    host = {n: torch.empty(p0[n].shape, dtype=p0[n].dtype, pin_memory=True).copy_(p0[n]) for n in names}
    devb = [{n: torch.empty_like(p0[n]) for n in names} for _ in range(2)]
    o = [o_buf[: L * T * H * dv].view(L, T, H, dv), torch.empty(L, T, H, dv, dtype=torch.float32, device=dev)]
    pi = [path_idx, torch.empty_like(path_idx)]
    pl = [path_len, torch.empty_like(path_len)]
    nt = [next_tok, torch.empty_like(next_tok)]
    o_host = torch.empty(o[0].shape, dtype=torch.float32, pin_memory=True)
    pi_host = torch.empty(path_idx.shape, dtype=torch.int32, pin_memory=True)
    pl_host = torch.empty(path_len.shape, dtype=torch.int32, pin_memory=True)
    nt_host = torch.empty(next_tok.shape, dtype=torch.int32, pin_memory=True)
    h2d = sum(host[n].numel() * host[n].element_size() for n in names)
    d2h = sum(x.numel() * x.element_size() for x in (o_host, pi_host, pl_host, nt_host))
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_done = [torch.cuda.Event() for _ in range(2)]      # kernels of the step using buffer set j have finished
    ev_out = [torch.cuda.Event() for _ in range(2)]       # results of buffer set j have reached the host

    def one(i):
        j = i & 1
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_done[j])                   # the step two back no longer reads these inputs
            for n in names:
                devb[j][n].copy_(host[n], non_blocking=True)
            ev_in[j].record(s_in)
        stream.wait_event(ev_in[j])
        stream.wait_event(ev_out[j])                      # its results have been read back
        d = devb[j]
        speca.verify_tree(dims, S, d["q"], d["k"], d["v"], d["alpha"], d["beta"], d["d_offs"], T, d["d_parent"],
                          d["d_depth"], o[j], None, ws, status)
        speca.greedy_accept(B, 8, d["d_offs"], d["d_parent"], d["d_draft"], d["d_target"], d["d_root"], pi[j], pl[j],
                            nt[j], status)
        speca.commit(dims, S, d["k"], d["v"], d["alpha"], d["beta"], d["d_offs"], T, d["d_parent"], pi[j], pl[j], status)
        ev_done[j].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[j])
            o_host.copy_(o[j], non_blocking=True)
            pi_host.copy_(pi[j], non_blocking=True)
            pl_host.copy_(pl[j], non_blocking=True)
            nt_host.copy_(nt[j], non_blocking=True)
            ev_out[j].record(s_out)

    for j in range(2):
        ev_done[j].record(stream)
        ev_out[j].record(stream)
    one(0)
    one(1)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = max(2, args.e2e_steps)
    e0.record(stream)
    for i in range(n):
        one(i)
    stream.wait_stream(s_out)
    stream.wait_stream(s_in)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    return {"value": T * L / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": n,
            "note": "draft inputs from pinned host memory, outputs and accepted paths read back, every step; uploads, "
                    "kernels and read-backs of consecutive steps overlap on three streams; state stays in HBM"}


# ---------------------------------------------------------------------------
# the oracle on the host cores (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------
def oracle_sample_problem(workload: str, H: int, dk: int, dv: int, n_units: int, seed: int = 4242):
    """A bounded sample of the workload: n_units (layer, sequence, head) units, half chains and half
    trees for cfg5 (ragged trees for cfg4), repacked as independent single-head sequences."""
    from paper_2607_16673_b200 import synth
    rng = np.random.default_rng(seed)
    parents = workload_parents(workload, rng, n_units)
    return synth.make_problem(seed, 1, 1, dk, dv, parents)


def time_oracle_once(prob):
    import oracle
    t0 = time.perf_counter()
    oracle.verify_tree(prob.S0, prob.q, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets, prob.parent)
    pi, pl, nt = oracle.greedy_accept(prob.node_offsets, prob.parent, prob.draft_tok, prob.target_tok,
                                      prob.root_target_tok, prob.max_depth)
    oracle.commit(prob.S0, prob.k, prob.v, prob.alpha, prob.beta, prob.node_offsets, pi, pl)
    return time.perf_counter() - t0


def cpu_baseline(workload: str, L: int, H: int, dk: int, dv: int, n_units: int = 1536, passes: int = 12):
    import oracle
    prob = oracle_sample_problem(workload, H, dk, dv, n_units)
    time_oracle_once(oracle_sample_problem(workload, H, dk, dv, 8))      # build + page in
    dt = sum(time_oracle_once(prob) for _ in range(passes))
    # one unit is 1/H of a token-layer
    value = passes * prob.T / H / dt
    # the same oracle on one thread, on a sixteenth of the sample
    small = oracle_sample_problem(workload, H, dk, dv, max(8, n_units // 16), seed=4343)
    cores = oracle.num_threads()
    prev_env = os.environ.get("OMP_NUM_THREADS")
    single = None
    try:
        oracle.set_num_threads(1)
        t1 = time_oracle_once(small)
        single = small.T / H / t1
    except AttributeError:
        pass
    finally:
        if hasattr(oracle, "set_num_threads"):
            oracle.set_num_threads(cores)
    return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "single_thread_value": single,
            "sample": f"{passes} passes over {n_units} (layer, sequence, head) units of {workload} ({prob.T} node-units "
                      f"per pass), verify+accept+commit, {dt:.1f} s of CPU work, scaled by 1/heads to token-layers"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    L, B, H, dk, dv, desc = WORKLOADS[args.workload]
    n_units = 192
    prob = oracle_sample_problem(args.workload, H, dk, dv, n_units)
    for _ in range(max(1, min(args.warmup, 3))):
        time_oracle_once(oracle_sample_problem(args.workload, H, dk, dv, 8))
    K = args.steps
    t = 0.0
    for _ in range(K):
        t += time_oracle_once(prob)
    value = K * prob.T / H / t
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
        "warmup": args.warmup, "ms_per_step": t / K * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {desc}", "sample_units_per_step": n_units},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": f"each step: {n_units} (layer, sequence, head) units of {args.workload} "
                                   f"({prob.T} node-units), scaled by 1/heads to token-layers"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------
# the paper's own target shape (h_v = 8, d_k = d_v = 256, 24 layers, one sequence) on the
# proposal shapes of Table 1: tree verification against root-to-leaf replay
# ---------------------------------------------------------------------------
PAPER_SHAPES = [(2, 12, 16), (2, 24, 32), (4, 4, 16), (4, 4, 32), (4, 12, 16), (4, 24, 32)]     # top-k, depth, nodes


def run_paper_shapes(args):
    """Per proposal shape: one tree verification of all 24 layers, against replaying every root-to-leaf
    path as its own chain (which recomputes shared prefixes and re-reads the state per path), and the
    commit of one accepted path.  The 48 MiB state would sit in L2, so eight copies are rotated."""
    import torch
    from paper_2607_16673_b200 import binding as speca
    from paper_2607_16673_b200 import synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    L, H, dk, dv, COPIES = args.layers or 24, 8, 256, 256, 8
    stream = torch.cuda.current_stream()
    rows = []
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    bf = lambda a: t(a.view(np.int16)).view(torch.bfloat16)

    def timed(fn, n=args.steps):
        for i in range(max(3, args.warmup)):
            fn(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(n):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    for (top_k, depth, nodes) in PAPER_SHAPES:
        rng = np.random.default_rng(1000 * top_k + 10 * depth + nodes)
        par = synth.proposal_tree_parent(top_k, depth, nodes, rng, 16)      # the library takes depth <= 16
        prob = synth.make_problem(77 + nodes + top_k, L, H, dk, dv, [par], max_depth=16)
        n = len(par)
        tree_depth = int(synth.depth_of(par).max())
        md = 8 if tree_depth <= 8 else 16            # depth <= 8 and <= 32 nodes: the tensor-core route applies
        dims = speca.Dims(L, 1, H, dk, dv, 1.0, md, 32, args.route)
        S = [t(prob.S0) + 0 for _ in range(COPIES)]
        q, k, v, al, be = bf(prob.q), bf(prob.k), bf(prob.v), t(prob.alpha), t(prob.beta)
        offs, parent = t(prob.node_offsets), t(prob.parent)
        o = torch.empty(L, n, H, dv, device=dev)
        ws = speca.alloc_workspace(dims, n, dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        ms_tree = timed(lambda i: speca.verify_tree(dims, S[i % COPIES], q, k, v, al, be, offs, n, parent, None, o, None,
                                                    ws, status))
        # root-to-leaf replay: one chain per leaf, each from its own copy of the state
        has_child = np.zeros(n, dtype=bool)
        has_child[par[par >= 0]] = True
        paths = [synth.root_path(par, int(leaf)) for leaf in np.flatnonzero(~has_child)]
        idx = np.concatenate(paths)
        offs_r = np.concatenate([[0], np.cumsum([len(p) for p in paths])]).astype(np.int32)
        Br, Tr = len(paths), int(offs_r[-1])
        dims_r = speca.Dims(L, Br, H, dk, dv, 1.0, md, 32, args.route)
        Sr = [S[c].expand(L, Br, H, dv, dk).contiguous() for c in range(2)]
        take = lambda x: x[:, t(idx).long()].contiguous()
        qr, kr, vr, alr, ber = take(q), take(k), take(v), take(al), take(be)
        o_r = torch.empty(L, Tr, H, dv, device=dev)
        ws_r = speca.alloc_workspace(dims_r, Tr, dev)
        ms_r2l = timed(lambda i: speca.verify_chain(dims_r, Sr[i % 2], qr, kr, vr, alr, ber, t(offs_r), Tr, o_r, None, ws_r,
                                                    status))
        # commit of the deepest path
        path = max(paths, key=len)[:8]
        pidx = torch.full((1, md), -1, dtype=torch.int32, device=dev)
        pidx[0, :len(path)] = t(np.asarray(path, np.int32))
        plen = torch.tensor([len(path)], dtype=torch.int32, device=dev)
        ms_commit = timed(lambda i: speca.commit(dims, S[i % COPIES], k, v, al, be, offs, n, parent, pidx, plen, status))
        # the whole round (verify -> accept -> commit), launched kernel by kernel and replayed as ONE CUDA graph:
        # at this size the round is launch-bound, and the entry points are capturable (no allocation, no
        # synchronisation, all arguments fixed at capture)
        draft, target, root = t(prob.draft_tok), t(prob.target_tok), t(prob.root_target_tok)
        gp = torch.full((1, md), -1, dtype=torch.int32, device=dev)
        gl = torch.zeros(1, dtype=torch.int32, device=dev)
        gn = torch.zeros(1, dtype=torch.int32, device=dev)

        def round_(i):
            speca.verify_tree(dims, S[i % COPIES], q, k, v, al, be, offs, n, parent, None, o, None, ws, status)
            speca.greedy_accept(1, md, offs, parent, draft, target, root, gp, gl, gn, status)
            speca.commit(dims, S[i % COPIES], k, v, al, be, offs, n, parent, gp, gl, status)

        ms_round = timed(round_)
        graphs = []
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            for c in range(COPIES):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    round_(c)
                graphs.append(g)
        stream.wait_stream(side)
        ms_graph = timed(lambda i: graphs[i % COPIES].replay())
        assert int(status.item()) == 0
        rows.append({"top_k": top_k, "config_depth": depth, "nodes": n, "tree_depth": tree_depth,
                     "round_ms": ms_round, "round_cuda_graph_ms": ms_graph,
                     "leaves": Br, "replayed_tokens": Tr, "verify_tree_ms": ms_tree, "r2l_replay_ms": ms_r2l,
                     "tree_vs_r2l": ms_r2l / ms_tree, "commit_ms": ms_commit, "accepted_len": len(path),
                     "token_layers_per_s": n * L / ((ms_tree + ms_commit) * 1e-3)})
    tot_tok = sum(r["nodes"] for r in rows) * L
    tot_ms = sum(r["verify_tree_ms"] + r["commit_ms"] for r in rows)
    print(json.dumps({
        "metric": METRIC, "value": tot_tok / (tot_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": tot_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "paper: 1 sequence x 24 layers x 8 heads, d_k=d_v=256 (the paper's target shape); the six "
                               "proposal shapes of Table 1 (top-k, configured depth, nodes), one verify + one commit each",
                   "l2": f"{COPIES} rotating copies of the 48 MiB state (larger than L2)", "route": args.route},
        "shapes": rows,
        "note": "latency-bound (192 units on 148 SMs); the paper's R2L column (19-91 ms on H100, whole target body) "
                "is context only: r2l_replay_ms here replays the recurrent layer alone through speca_verify_chain"}))



# ---------------------------------------------------------------------------
# the two small single-sequence configurations (latency-bound: 384 units on 148 SMs, 24 MiB of state)
# ---------------------------------------------------------------------------
def run_small(args):
    """cfg2: 1 sequence x 24 layers x 16 heads, d_k = d_v = 128, a chain of 8 draft tokens, accepted length drawn
    uniformly from 0..8 per step, beside the same 8 tokens by 8 speca_decode_step calls.  cfg3: the same shape with a
    32-node tree (depth <= 6) and a random root-to-leaf accepted path.  The 24 MiB state fits L2, so eight copies
    are rotated (192 MiB, larger than L2) and the L2-resident figure (one copy) is reported beside it.  Also
    reported: what one call costs the host (enqueue time with the GPU kept busy)."""
    import torch
    from paper_2607_16673_b200 import binding as speca
    from paper_2607_16673_b200 import synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream()
    L, H, dk, dv, COPIES = args.layers or 24, 16, 128, 128, 8
    chain = args.workload == "cfg2"
    rng = np.random.default_rng(2 if chain else 3)
    par = synth.chain_parent(8) if chain else synth.random_tree_parent(32, 6, 4, rng)
    n = len(par)
    prob = synth.make_problem(20 + n, L, H, dk, dv, [par], max_depth=8)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    bf = lambda a: t(a.view(np.int16)).view(torch.bfloat16)
    dims = speca.Dims(L, 1, H, dk, dv, 1.0, 8, 8 if chain else 32, args.route)
    S = [t(prob.S0) + 0 for _ in range(COPIES)]
    q, k, v, al, be = bf(prob.q), bf(prob.k), bf(prob.v), t(prob.alpha), t(prob.beta)
    offs, parent = t(prob.node_offsets), t(prob.parent)
    draft, target, root = t(prob.draft_tok), t(prob.target_tok), t(prob.root_target_tok)
    o = torch.empty(L, n, H, dv, device=dev)
    ws = speca.alloc_workspace(dims, n, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    # accepted paths: cfg2 a prefix of length 0..8 per step, cfg3 a random root-to-leaf path
    NP = 16
    has_child = np.zeros(n, dtype=bool)
    has_child[par[par >= 0]] = True
    leaves = np.flatnonzero(~has_child)
    paths_h = [list(range(int(rng.integers(0, 9)))) if chain else synth.root_path(par, int(rng.choice(leaves)))
               for _ in range(NP)]
    pidx = [torch.full((1, 8), -1, dtype=torch.int32, device=dev) for _ in range(NP)]
    plen = [torch.tensor([len(p_)], dtype=torch.int32, device=dev) for p_ in paths_h]
    for j, p_ in enumerate(paths_h):
        if p_:
            pidx[j][0, :len(p_)] = t(np.asarray(p_, np.int32))
    gp = torch.full((1, 8), -1, dtype=torch.int32, device=dev)
    gl = torch.zeros(1, dtype=torch.int32, device=dev)
    gn = torch.zeros(1, dtype=torch.int32, device=dev)

    def verify(Sx):
        if chain:
            speca.verify_chain(dims, Sx, q, k, v, al, be, offs, n, o, None, ws, status)
        else:
            speca.verify_tree(dims, Sx, q, k, v, al, be, offs, n, parent, None, o, None, ws, status)

    def step(i, copies):
        Sx = S[i % copies]
        verify(Sx)
        speca.greedy_accept(1, 8, offs, parent, draft, target, root, gp, gl, gn, status)
        speca.commit(dims, Sx, k, v, al, be, offs, n, parent, pidx[i % NP], plen[i % NP], status)

    def timed(fn, reps):
        for i in range(max(3, args.warmup)):
            fn(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        w0 = time.perf_counter()
        e0.record(stream)
        for i in range(reps):
            fn(i)
        e1.record(stream)
        w1 = time.perf_counter()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps, (w1 - w0) / reps * 1e6

    K = max(args.steps, 20)
    sampler = ClockSampler(0)
    sampler.mark()
    ms_step, _ = timed(lambda i: step(i, COPIES), K)
    sampler.mark()
    clocks = sampler.stop()
    ms_step_l2, _ = timed(lambda i: step(i, 1), K)
    def host_us(fn, reps=50):
        """Wall time the host spends inside one call, the GPU idle beforehand (so the launch queue never blocks)."""
        tot = 0.0
        for i in range(reps + 5):
            torch.cuda.synchronize()
            w0 = time.perf_counter()
            fn(i)
            w1 = time.perf_counter()
            if i >= 5:
                tot += w1 - w0
        torch.cuda.synchronize()
        return tot / reps * 1e6

    ms_verify, _ = timed(lambda i: verify(S[i % COPIES]), K)
    us_verify_host = host_us(lambda i: verify(S[i % COPIES]))
    ms_verify_l2, _ = timed(lambda i: verify(S[0]), K)
    commit_fn = lambda i: speca.commit(dims, S[i % COPIES], k, v, al, be, offs, n, parent, pidx[i % NP], plen[i % NP], status)
    ms_commit, _ = timed(commit_fn, K)
    us_commit_host = host_us(commit_fn)
    # the same tokens one at a time: n decode steps (chain order; for the tree, its first root-to-leaf path)
    d1 = speca.Dims(L, 1, H, dk, dv)
    order = list(range(n)) if chain else paths_h[0]
    qs = [q[:, j:j + 1].contiguous() for j in order]
    ks = [k[:, j:j + 1].contiguous() for j in order]
    vs = [v[:, j:j + 1].contiguous() for j in order]
    als = [al[:, j:j + 1].contiguous() for j in order]
    bes = [be[:, j:j + 1].contiguous() for j in order]
    o1 = torch.empty(L, 1, H, dv, device=dev)

    def decode_all(i):
        Sx = S[i % COPIES]
        for j in range(len(order)):
            speca.decode_step(d1, Sx, qs[j], ks[j], vs[j], als[j], bes[j], o1)

    ms_decode, _ = timed(decode_all, K)
    assert int(status.item()) == 0
    mean_acc = float(np.mean([len(p_) for p_ in paths_h]))
    Sb = 4 * dk * dv
    units = L * H
    vbytes = units * Sb + n * units * (4 * dk + 2 * dv + 8 + 4 * dv)
    cbytes = 2 * units * Sb * float(np.mean([len(p_) > 0 for p_ in paths_h])) + mean_acc * units * (2 * dk + 2 * dv + 8)
    peak, peak_kind = measured_peak_gbs()
    achieved = (vbytes + cbytes) / (ms_step * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": n * L / (ms_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K,
        "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: 1 seq x {L} layers x {H} heads, d_k=d_v=128; " +
                               ("chain of 8, accepted length uniform 0..8" if chain else
                                f"{n}-node tree (depth {int(synth.depth_of(par).max())}), random root-to-leaf path"),
                   "l2": f"{COPIES} rotating copies of the {units * Sb / 2**20:.0f} MiB state (larger than L2)",
                   "route": args.route, "mean_accepted_len": mean_acc},
        "roofline": {"bound": "hbm", "kernel": "step", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                     "note": "latency-bound: 384 units on 148 SMs, a few tens of MB per call"},
        "latency_ms": {"step": ms_step, "step_l2_resident": ms_step_l2, "plan_verify": ms_verify,
                       "plan_verify_l2_resident": ms_verify_l2, "commit": ms_commit,
                       "same_tokens_by_decode_steps": ms_decode, "decode_steps": len(order)},
        "host_us_per_call": {"verify": us_verify_host, "commit": us_commit_host,
                             "note": "wall time of one call on the host (Python binding + C entry point: argument checks, tensor maps, "
                                     "launches), GPU idle beforehand"},
        "gpu_launches": (3 if chain and args.route == 1 else 4) * K,
        "clocks": clocks,
    }
    print(json.dumps(out))


# ---------------------------------------------------------------------------
# sweeps behind the figures in the design doc
# ---------------------------------------------------------------------------
def run_sweep(args):
    import torch
    from paper_2607_16673_b200 import binding as speca
    from paper_2607_16673_b200 import synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream()
    L, B, H, dk, dv = args.layers or 24, args.batch or 128, 16, 128, 256
    peak, peak_kind = measured_peak_gbs()
    t = lambda a: torch.from_numpy(a).to(dev)

    def timed(fn, reps=10):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    S = synth.device_state(1, L, B, H, dk, dv, 0.02, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rows = []
    if args.sweep == "commit-len":
        # every sequence an 8-token chain, the first A tokens accepted
        hi = host_round_inputs("chains8", B, 5000)
        q, k, v, al, be = synth.device_records(7, L, hi["T"], H, dk, dv, dev)
        dims = speca.Dims(L, B, H, dk, dv, 1.0, 8, 64, args.route)
        offs, par = t(hi["node_offsets"]), t(hi["parent"])
        for A in (1, 2, 3, 4, 5, 6, 8):
            pidx = torch.arange(8, dtype=torch.int32, device=dev).repeat(B, 1).contiguous()
            plen = torch.full((B,), A, dtype=torch.int32, device=dev)
            ms = timed(lambda: speca.commit(dims, S, k, v, al, be, offs, hi["T"], par, pidx, plen, status))
            nbytes = 2 * L * B * H * 4 * dk * dv + A * B * L * H * (2 * dk + 2 * dv + 8)
            rows.append({"accepted": A, "ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "frac": nbytes / (ms * 1e-3) / 1e9 / peak})
    elif args.sweep == "role-waits":
        # Per-role wait cycles of the tensor-core verification, recorded by CTA 0 of a library built with -DSPECA_PROF
        # (SPECA_NVCC_FLAGS=-DSPECA_PROF python -m paper_2607_16673_b200.build --force): for one warp of every role its
        # lifetime in cycles and the share of it spent in each of up to eight kinds of wait or code segment (the slot
        # numbers are the first argument of the WAIT / PROF_SEG macros in the kernel source).  The instrumented build
        # is 20-40 % slower than the plain one: read the shares, not the times.
        if not speca.lib().speca_test_profiling_build():
            print(json.dumps({"sweep": args.sweep, "error": "library not built with -DSPECA_PROF: rebuild with "
                              "SPECA_NVCC_FLAGS=-DSPECA_PROF python -m paper_2607_16673_b200.build --force"}))
            return
        L = args.layers or 4
        S = synth.device_state(1, L, B, H, dk, dv, 0.02, dev)
        roles = {0: {0: "TMA producer", 1: "MMA issuer, tile 0", 14: "MMA issuer, tile 1", 2: "preparation", 6: "epilogue group 0",
                     10: "epilogue group 1", 15: "split"},
                 3: {0: "TMA producer", 1: "MMA issuer", 2: "preparation", 6: "epilogue group 0", 10: "epilogue group 1"},
                 4: {0: "TMA producer", 1: "first pass, tile 0", 18: "first pass, tile 1", 19: "correction, tile 0",
                     20: "correction, tile 1", 2: "solver", 6: "vector", 10: "split", 14: "epilogue"}}
        sm = torch.cuda.get_device_properties(dev).multi_processor_count
        for wl in ("chains8", "trees64", "cfg5"):
            hi = host_round_inputs(wl, B, 5000)
            q, k, v, al, be = synth.device_records(7, L, hi["T"], H, dk, dv, dev)
            offs, par = t(hi["node_offsets"]), t(hi["parent"])
            o = torch.empty(L, hi["T"], H, dv, device=dev)
            dims = speca.Dims(L, B, H, dk, dv, 1.0, 8, 64, args.route)
            ws = speca.alloc_workspace(dims, hi["T"], dev)
            ms = timed(lambda: speca.verify_tree(dims, S, q, k, v, al, be, offs, hi["T"], par, None, o, None, ws, status), reps=1)
            ctrl = ws[:2048].cpu().numpy().view(np.int64)
            for w, name in roles.get(args.route, roles[0]).items():
                vals = ctrl[8 + w * 9: 8 + w * 9 + 9]
                if vals[8] > 0:
                    rows.append({"units": wl, "warp": w, "role": name, "life_kcycles": float(vals[8]) / 1e3,
                                 "share_pct": [round(100.0 * float(x) / float(vals[8]), 1) for x in vals[:8]]})
            rows.append({"units": wl, "verify_ms": ms, "us_per_unit_per_sm": ms * 1e3 / (L * B * H / sm)})
    else:
        sm = torch.cuda.get_device_properties(dev).multi_processor_count
        for wl in ("chains8", "trees64"):
            hi = host_round_inputs(wl, B, 5000)
            q, k, v, al, be = synth.device_records(7, L, hi["T"], H, dk, dv, dev)
            offs, par = t(hi["node_offsets"]), t(hi["parent"])
            o = torch.empty(L, hi["T"], H, dv, device=dev)
            for name, route in (("default (fp32-grade)", 0), ("single-pass TF32", 3), ("effective-query", 4)):
                dims = speca.Dims(L, B, H, dk, dv, 1.0, 8, 64, route)
                ws = speca.alloc_workspace(dims, hi["T"], dev)
                ms = timed(lambda: speca.verify_tree(dims, S, q, k, v, al, be, offs, hi["T"], par, None, o, None, ws, status))
                nbytes = L * B * H * 4 * dk * dv + hi["T"] * L * H * (4 * dk + 2 * dv + 8 + 4 * dv)
                rows.append({"units": wl, "route": name, "verify_ms": ms, "us_per_unit_per_sm": ms * 1e3 / (L * B * H / sm),
                             "gbs": nbytes / (ms * 1e-3) / 1e9, "frac": nbytes / (ms * 1e-3) / 1e9 / peak})
    assert int(status.item()) == 0
    print(json.dumps({"sweep": args.sweep, "shape": f"{B} seq x {L} layers x {H} heads, d_k={dk} d_v={dv}",
                      "peak_gbs": peak, "peak_kind": peak_kind, "rows": rows}))


def spawn_ranks(args):
    """`python bench.py --gpus N` outside a launcher: start N ranks of this script, one process per GPU."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)
def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(spawn_ranks(args))
    if args.sweep and args.impl != "reference":
        run_sweep(args)
        return
    if args.workload in ("cfg2", "cfg3") and args.impl != "reference":
        run_small(args)
        return
    if args.workload == "paper" and args.impl != "reference":
        run_paper_shapes(args)
        return
    if args.impl == "reference" and args.workload in ("paper", "cfg2", "cfg3"):
        args.workload = "cfg5"
    if args.impl == "reference":
        run_reference(args)
    else:
        run_speca(args)


if __name__ == "__main__":
    main()
