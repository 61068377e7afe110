"""The N > 1 path of the benchmark on CPU (gloo, world_size 2): ranks take independent batches, the
job time is the max over ranks, only rank 0 reports; and `--impl reference` under torchrun."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    import mdn_workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.Workload("t", B=1, T=64, H=1, dk=64, dv=64, dtype="f32")
    wr = bench.rank_workload(w, rank)
    q = wl.make_inputs(wr)["q"]
    elapsed = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")      # rank 1 is the slow one
    value = bench.job_tokens_per_s(w, world, 3, elapsed)
    gathered = [None] * world
    dist.all_gather_object(gathered, float(np.abs(q).sum()))
    if rank == 0:
        out.put((wr.seed, elapsed, value, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_ranks_are_independent_batches_and_time_is_max_over_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 400
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    seed0, elapsed, value, sums = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert seed0 == 0 and elapsed == 15.0
    assert abs(value - 64 * 2 * 3 / 15e-3) < 1e-6
    assert sums[0] != sums[1]            # different data on each rank


def test_reference_arm_under_torchrun_prints_one_line_from_rank0():
    port = 29900 + os.getpid() % 90
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--config", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] == 0
