"""Host logic of the N > 1 path, on CPU with the gloo backend (world size 2): the batch is
partitioned over ranks with no data-path collective; only the timing/size bookkeeping is reduced
(MAX of times, SUM of work), and only rank 0 reports."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r pretends to have taken (10 + r) ms for (100 + r) tokens
    res = bench.reduce_over_ranks(dist, torch.device("cpu"), 10.0 + rank, 6.0 - rank, 3.0 + 2 * rank,
                                  100 + rank, 1000 * (rank + 1), 500)
    # every rank draws its own sequences
    topo = bench.host_round_inputs("cfg5", 8, bench.rank_seed(5000, rank, 0))
    gathered = [None] * world
    dist.all_gather_object(gathered, topo["parent"].tolist())
    if rank == 0:
        out.put((res, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_max_time_and_sum_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    total_ms, t_verify, t_commit, tokens, vb, cb = res
    assert (total_ms, t_verify, t_commit) == (11.0, 6.0, 5.0)          # max over ranks
    assert (tokens, vb, cb) == (201.0, 3000.0, 1000.0)                  # sum over ranks
    assert gathered[0] != gathered[1]                                    # different sequences per rank


def test_rank_seeds_are_distinct():
    seeds = {bench.rank_seed(base, r, j) for base in (1000, 5000, 7000) for r in range(8) for j in range(bench.POOL)}
    assert len(seeds) == 3 * 8 * bench.POOL


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "1", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "1", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0


def test_algorithmic_bytes_formula():
    """Byte counts of one step at the benchmark configuration (d_k=128, d_v=256, 24 layers, 16 heads)."""
    L, B, H, dk, dv, T = 24, 128, 16, 128, 256, 4608
    path_len = np.array([2] * 100 + [0] * 28)
    v, c = bench.algorithmic_bytes(L, B, H, dk, dv, T, path_len)
    units, Sb = L * B * H, 4 * dk * dv
    assert v == units * Sb + T * L * H * (4 * dk + 2 * dv + 8) + T * L * H * 4 * dv == 10080485376
    assert c == 2 * 100 * L * H * Sb + 200 * L * H * (2 * dk + 2 * dv + 8)


def test_gpus_flag_starts_one_rank_per_gpu(monkeypatch):
    """`python bench.py --gpus N` outside a launcher re-executes itself under torch.distributed.run with N ranks on
    127.0.0.1; inside a launcher (WORLD_SIZE set) it must not spawn again."""
    calls = []
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: calls.append(cmd) or 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "1"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    with pytest.raises(SystemExit) as e:
        bench.main()
    assert e.value.code == 0 and len(calls) == 1
    cmd = calls[0]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "2", "--steps", "1"] and os.path.basename(cmd[-5]) == "bench.py"


def test_launcher_runs_two_ranks_end_to_end_on_cpu():
    """The same launch line the multi-GPU benchmark uses, with the arm that needs no GPU: two ranks start, rank 0
    prints the one JSON line, rank 1 exits 0 without output."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                        "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
                        "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1"],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2


def test_traffic_table_is_read_per_workload_kernel_and_route():
    """roofline.traffic comes from the table of ncu captures under profiles/: captured bytes x scale, None if absent."""
    import bench
    v = bench.ncu_traffic("cfg5", "verify")
    c = bench.ncu_traffic("cfg5", "commit")
    assert v is not None and c is not None
    # one launch streams the 6.4 GB state once (verify) or twice (commit) plus records and outputs
    assert 8e9 < v < 12e9 and 7e9 < c < 14e9
    assert bench.ncu_traffic("cfg5-tf32", "verify") is not None
    assert bench.ncu_traffic("cfg5", "no such kernel") is None and bench.ncu_traffic("nothing", "verify") is None


def test_test_only_symbols_are_exported_but_not_declared():
    """The switches the tests use are reachable through the library, not through the public header."""
    import ctypes
    import os
    from paper_2607_16673_b200 import binding
    header = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "speca.h")).read()
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in ("speca_test_withhold_first_load", "speca_test_commit_long_min_tiles", "speca_test_profiling_build"):
        assert hasattr(lib, name) and name not in header
    assert lib.speca_test_profiling_build() == 0, "the committed build configuration carries no profiling counters"
