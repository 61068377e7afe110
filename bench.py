#!/usr/bin/env python
"""Benchmark of the MDN chunkwise forward (one "step" = one mdn_chunk_fwd call = the whole hot
path: chunk map, coefficient scan, intra-chunk solve, inter-chunk propagation, output).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

Prints ONE JSON line.  Metric: tokens/s of the forward on the 1.3B-layer-shaped workload
(B=8, H=16, T=4096, dk=dv=128, bf16), inputs resident in HBM.  N > 1 (torchrun): every rank
runs its own batch of the same shape (batches are independent: no data-path collective);
value = all ranks' tokens / max-over-ranks time ("weak" scaling).

`--impl reference` times the fp64 CPU oracle (the only CPU code in this repository) on a
bounded sample of the same workload; it is a deliberately slow program, reported for context.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import mdn_workloads as wl  # noqa: E402

METRIC = "MDN chunkwise fwd tokens/s"
UNIT = "tokens/s"
BYTES_PER_HEAD_TOKEN_BF16 = 1040      # q,k,v read + o written (bf16, d=128) + four fp32 gates
L2_BYTES = 126e6
# dram__bytes_read.sum + dram__bytes_write.sum per launch come from the ncu summaries under profiles/ (same command
# line as this benchmark): each summary carries the lines "kernel = <name>", "workload = <name>" and
# "traffic_bytes_per_launch = <bytes>", which are read at run time, so the number cannot drift away from its source.
PROFILE_FILES = {"chain": "chain_tf32_cfg2.md", "intra_chunk": "intra_mma_cfg2.md"}
STAGE_KERNELS = {"chain": "chain_tf32_kernel", "intra_chunk": "intra_mma_kernel"}


def profile_traffic(stage: str, workload: str):
    """(bytes per launch, source) from the committed ncu summary of this stage's kernel on this workload, or
    (None, reason) when there is no summary of exactly that kernel and workload."""
    import re
    name = PROFILE_FILES.get(stage)
    path = os.path.join(ROOT, "profiles", name) if name else None
    if not path or not os.path.exists(path):
        return None, "no ncu summary for stage %r" % stage
    text = open(path).read()
    fields = dict(re.findall(r"^(kernel|workload|traffic_bytes_per_launch)\s*=\s*(\S+)\s*$", text, flags=re.M))
    if fields.get("kernel") != STAGE_KERNELS[stage] or fields.get("workload") != workload:
        return None, "profiles/%s covers %s on %s" % (name, fields.get("kernel"), fields.get("workload"))
    src = {"file": "profiles/" + name, "commit": git_hash(["log", "-1", "--format=%h", "--", "profiles/" + name])}
    return float(fields["traffic_bytes_per_launch"]), src


def git_hash(args=("rev-parse", "--short", "HEAD")):
    """Short hash from git, else from the stamp the build step leaves beside the library (the GPU machine gets no .git)."""
    try:
        out = subprocess.run(["git", "-C", ROOT] + list(args), capture_output=True, text=True, timeout=10)
        if out.returncode == 0 and out.stdout.strip():
            return out.stdout.strip()
    except (OSError, subprocess.SubprocessError):
        pass
    try:
        info = json.load(open(os.path.join(ROOT, "paper_2605_05838_b200", "_build_info.json")))
        return info.get("git_hash") if list(args) == ["rev-parse", "--short", "HEAD"] else info.get("profiles", {}).get(args[-1])
    except (OSError, ValueError):
        return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def workload_desc(w: wl.Workload) -> str:
    kind = "packed varlen" if w.varlen else "fixed length"
    return "%s: B=%d,H=%d,T=%d,dk=%d,dv=%d,%s,chunk=64,%s" % (w.name, w.B, w.H, w.T, w.dk, w.dv, w.dtype, kind)


def algorithmic_bytes(w: wl.Workload, n_state: int, has_init: bool) -> float:
    es = 2 if w.dtype == "bf16" else 4
    per_ht = es * (2 * w.dk + 2 * w.dv) + 16
    states = n_state * w.H * w.dk * w.dv * 4 * (2 + (2 if has_init else 0))
    return float(w.B * w.T * w.H * per_ht + states)


def algorithmic_flops(w: wl.Workload) -> float:
    return float(w.B * w.T * w.H) * (12 * w.dk * w.dv + 4 * 64 * (w.dk + w.dv))


def rank_workload(w: wl.Workload, rank: int) -> wl.Workload:
    """Every rank runs its own batch of the same shape (seed offset by rank): batches are independent
    problems, so there is no data-path collective."""
    import dataclasses
    return dataclasses.replace(w, seed=w.seed + rank)


def max_over_ranks(value: float, dist, device) -> float:
    """Max of a per-rank scalar over all ranks (the job's time is its slowest rank's)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(w: wl.Workload, world: int, steps: int, elapsed_ms: float) -> float:
    """Whole-job throughput: all ranks' tokens over the max-over-ranks time."""
    return w.B * w.T * world * steps / (elapsed_ms * 1e-3)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples during the timed region (reading only)."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "20"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def oracle_sample_tokens_per_s(w: wl.Workload, inp, target_s: float):
    """Times the oracle as it stands on a subset of (sequence, head) chains of this workload.
    Returns (tokens/s, threads, description, seconds)."""
    import oracle
    N = len(inp["seq_len"])
    total = N * w.H
    rng = np.random.default_rng(0)
    order = rng.permutation(total)

    def run(chains):
        t0 = time.perf_counter()
        oracle.stepwise(inp["q"], inp["k"], inp["v"], inp["beta"], inp["log_alpha"], inp["log_mu"], inp["eta"],
                        scale=inp["scale"], S0=inp["S0"], M0=inp["M0"], seq_start=inp["seq_start"],
                        seq_len=inp["seq_len"], chains=chains)
        return time.perf_counter() - t0

    def head_tokens(chains):
        return float(sum(int(inp["seq_len"][c // w.H]) for c in chains))

    threads = oracle.num_threads()
    probe = order[:min(total, max(threads, 4))]
    t_probe = run(probe)
    per_ht = t_probe / head_tokens(probe)
    want = int(min(total, max(len(probe), target_s / max(per_ht, 1e-12) / (head_tokens(order) / total))))
    chains = order[:want]
    secs = run(chains)
    ht = head_tokens(chains)
    # a token is all H heads: tokens/s = head-tokens/s / H
    return ht / w.H / secs, threads, "%d of %d (sequence, head) chains, %d head-tokens" % (len(chains), total, int(ht)), secs


def parity_report(mdn, w, inp, t, p, args, ws):
    """The timed workload's result against the oracle on EVERY (sequence, head) chain, outside any timed region:
    max |x - ref| / RMS(ref) of o as stored (bf16 on the bf16 workloads), of the oracle's own o rounded to that storage
    type (what one storage rounding of the exact result costs), of o stored as fp32 by the same kernels, and of
    the final states."""
    import oracle
    import torch
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import bf16_floor, rel_err
    t0 = time.perf_counter()
    o_ref, S_ref, M_ref = oracle.stepwise(inp["q"], inp["k"], inp["v"], inp["beta"], inp["log_alpha"], inp["log_mu"],
                                          inp["eta"], scale=inp["scale"], S0=inp["S0"], M0=inp["M0"],
                                          seq_start=inp["seq_start"], seq_len=inp["seq_len"])
    secs = time.perf_counter() - t0
    kw = dict(initial_S=t["initial_S"], initial_M=t["initial_M"], cu_seqlens=t["cu_seqlens"], scale=inp["scale"],
              path=args.path, workspace=ws)
    gates = (t["beta"], t["log_alpha"], t["log_mu"], t["eta"])
    o, S, M = mdn.chunk_fwd(t["q"], t["k"], t["v"], *gates, **kw)
    o32, _, _ = mdn.chunk_fwd(t["q"], t["k"], t["v"], *gates, o_dtype=torch.float32, **kw)
    torch.cuda.synchronize()
    f64 = lambda x: x.float().cpu().numpy().astype(np.float64)
    out = {"chains": int(len(inp["seq_len"]) * w.H), "oracle_seconds": secs,
           "o_stored": rel_err(f64(o), o_ref), "o_f32_store": rel_err(f64(o32), o_ref),
           "S": rel_err(f64(S), S_ref), "M": rel_err(f64(M), M_ref),
           "metric": "max |x - ref| / RMS(ref) over all elements", "tolerance": 2e-2 if w.dtype == "bf16" else 1e-4}
    if w.dtype == "bf16":
        out["o_bf16_floor"] = bf16_floor(o_ref)      # the exact result rounded once to bf16
    return out


def time_config(mdn, w, path, peaks):
    """ms per step of another named workload (device-resident inputs, CUDA events, 3 warm-up + 10 timed steps)."""
    import torch
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import to_torch
    inp = wl.make_inputs(w)
    t = to_torch(inp)
    N = len(inp["seq_len"])
    o_dtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    p = mdn.make_params(t["q"], t["v"], num_seqs=(N if w.varlen else 0), scale=inp["scale"], o_dtype=o_dtype, path=path)
    ws = torch.empty(mdn.workspace_bytes(p), dtype=torch.uint8, device=t["q"].device)
    io_bytes = algorithmic_bytes(w, N, t["initial_S"] is not None)
    n_copies = 1 if io_bytes > L2_BYTES else int(2 * L2_BYTES // io_bytes) + 1
    clone = lambda d: {k_: (v_.clone() if torch.is_tensor(v_) else v_) for k_, v_ in d.items()}
    sets = [t] + [clone(t) for _ in range(n_copies - 1)]
    outs = [torch.empty((w.B, w.T, w.H, w.dv), dtype=o_dtype, device=t["q"].device) for _ in range(n_copies)]

    def step(i):
        ti = sets[i % n_copies]
        mdn.chunk_fwd(ti["q"], ti["k"], ti["v"], ti["beta"], ti["log_alpha"], ti["log_mu"], ti["eta"],
                      initial_S=ti["initial_S"], initial_M=ti["initial_M"], cu_seqlens=ti["cu_seqlens"],
                      scale=inp["scale"], o_dtype=o_dtype, path=path, workspace=ws, out=outs[i % n_copies])

    for i in range(3):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(10):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / 10
    return {"workload": workload_desc(w), "ms_per_step": ms, "tokens_per_s": w.B * w.T / (ms * 1e-3),
            "frac": io_bytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "launches_per_step": mdn.last_launch_count(),
            "l2": "single copy" if n_copies == 1 else "%d copies rotated" % n_copies}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    inp = wl.make_inputs(w)
    N = len(inp["seq_len"])
    total = N * w.H
    threads = oracle.num_threads()
    chains = np.random.default_rng(0).permutation(total)[:min(total, 2 * max(threads, 4))]
    ht = float(sum(int(inp["seq_len"][c // w.H]) for c in chains))

    def step():
        oracle.stepwise(inp["q"], inp["k"], inp["v"], inp["beta"], inp["log_alpha"], inp["log_mu"], inp["eta"],
                        scale=inp["scale"], S0=inp["S0"], M0=inp["M0"], seq_start=inp["seq_start"],
                        seq_len=inp["seq_len"], chains=chains)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = ht / w.H * args.steps / dt
    sample = "each step: %d of %d (sequence, head) chains = %d head-tokens" % (len(chains), total, int(ht))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_desc(w), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_ours(args, w):
    import torch
    import paper_2605_05838_b200 as mdn
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import to_torch

    mdn.lib()   # fail loudly if the CUDA library is missing
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # the clock sampler starts before the inputs are generated (seconds of host work), so that nvidia-smi is already
    # sampling when the warm-up begins and the warm-up can be exactly what --warmup asks for
    sampler = ClockSampler(local) if rank == 0 else None
    wr = rank_workload(w, rank)
    inp = wl.make_inputs(wr)
    t = to_torch(inp, device="cuda:%d" % local)
    o_dtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    N = len(inp["seq_len"])
    p = mdn.make_params(t["q"], t["v"], num_seqs=(N if w.varlen else 0), scale=inp["scale"], o_dtype=o_dtype,
                        path=args.path)
    ws = torch.empty(mdn.workspace_bytes(p), dtype=torch.uint8, device=t["q"].device)
    # a workload whose inputs + outputs fit in the 126 MB L2 would be timed out of cache: rotate enough copies of
    # every input and of the output that one round exceeds twice the L2
    io_bytes = algorithmic_bytes(w, N, t["initial_S"] is not None)
    n_copies = 1 if io_bytes > L2_BYTES else int(2 * L2_BYTES // io_bytes) + 1
    clone = lambda d: {k_: (v_.clone() if torch.is_tensor(v_) else v_) for k_, v_ in d.items()}
    sets = [t] + [clone(t) for _ in range(n_copies - 1)]
    outs = [torch.empty((w.B, w.T, w.H, w.dv), dtype=o_dtype, device=t["q"].device) for _ in range(n_copies)]
    calls = [0]

    def step():
        i = calls[0] % n_copies
        calls[0] += 1
        ti = sets[i]
        return mdn.chunk_fwd(ti["q"], ti["k"], ti["v"], ti["beta"], ti["log_alpha"], ti["log_mu"], ti["eta"],
                             initial_S=ti["initial_S"], initial_M=ti["initial_M"], cu_seqlens=ti["cu_seqlens"],
                             scale=inp["scale"], o_dtype=o_dtype, path=args.path, workspace=ws, out=outs[i])

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    n_warm = max(args.warmup, 3)      # the timing rules ask for at least three
    for _ in range(n_warm):
        step()
    launches_per_step = mdn.last_launch_count()
    barrier()
    # timed region 1: exactly K steps, nothing but the calls -> the headline value
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(args.steps):
        step()
    ev1.record()
    barrier()
    elapsed_ms = ev0.elapsed_time(ev1)
    # timed region 2: K more steps with the library's per-stage events switched on (they serialise the
    # programmatic dependent launches a little, so they stay out of region 1) -> per-kernel durations
    stage_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(mdn.NUM_STAGE_EVENTS)] for _ in range(args.steps)]
    for i in range(args.steps):
        mdn.set_stage_events(stage_ev[i])
        step()
    mdn.set_stage_events(None)
    barrier()
    clocks = sampler.stop() if sampler else None
    elapsed_ms = max_over_ranks(elapsed_ms, dist, "cuda")
    tokens_per_step = w.B * w.T * world
    value = job_tokens_per_s(w, world, args.steps, elapsed_ms)

    # per-kernel durations, timed live; the roofline fraction is that of the WHOLE step (the path is two kernels in
    # series: algorithmic bytes over the time of one step); the dominant kernel's own figures are given beside it
    names = mdn.STAGE_NAMES
    stage_ms = {names[s]: statistics.mean(stage_ev[i][s].elapsed_time(stage_ev[i][s + 1]) for i in range(args.steps))
                for s in range(len(names))}
    dom = max(stage_ms, key=stage_ms.get)
    peaks = load_peaks()
    abytes = algorithmic_bytes(w, N, t["initial_S"] is not None)
    aflops = algorithmic_flops(w)
    step_s = elapsed_ms / args.steps * 1e-3
    dom_s = stage_ms[dom] * 1e-3
    achieved = abytes / step_s / 1e9
    tensor_path = mdn.resolved_path(p) == "tensor"
    traffic, sources = {}, {}
    for st_name in ("intra_chunk", "chain"):
        traffic[st_name], sources[st_name] = profile_traffic(st_name, w.name) if tensor_path else (None, "no summary for the SIMT path")
    whole_traffic = None if None in traffic.values() else sum(traffic.values())
    roofline = {"bound": "hbm", "kernel": "whole step: intra_chunk + chain (two kernels in series)", "achieved": achieved,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": whole_traffic,
                "traffic_source": sources, "peak_source": peaks["source"],
                "stage_ms": stage_ms, "algorithmic_bytes": abytes, "algorithmic_flops": aflops,
                "frac_of_nominal_hbm_8tbs": achieved / 8000.0,
                "tensor_achieved_tflops": aflops / step_s / 1e12,
                "tensor_frac_of_burst_peak": aflops / step_s / 1e12 / peaks["bf16_tflops"],
                "dominant_kernel": {"name": dom, "kernel_ms": stage_ms[dom], "traffic": traffic.get(dom),
                                    "frac_algorithmic_bytes_over_its_time": abytes / dom_s / 1e9 / peaks["hbm_gbs"],
                                    "tensor_achieved_tflops": aflops / dom_s / 1e12}}

    # end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        th = to_torch(inp, host_pinned=True)
        arena = torch.empty(mdn.host_arena_bytes(p), dtype=torch.uint8, device=t["q"].device)
        nst = N
        out = (torch.empty((w.B, w.T, w.H, w.dv), dtype=o_dtype).pin_memory(),
               torch.empty((nst, w.H, w.dk, w.dv), dtype=torch.float32).pin_memory(),
               torch.empty((nst, w.H, w.dk, w.dv), dtype=torch.float32).pin_memory())

        def e2e_step():
            mdn.chunk_fwd_host(th["q"], th["k"], th["v"], th["beta"], th["log_alpha"], th["log_mu"], th["eta"],
                               initial_S=th["initial_S"], initial_M=th["initial_M"], cu_seqlens=th["cu_seqlens"],
                               scale=inp["scale"], o_dtype=o_dtype, path=args.path, arena=arena, out=out)

        e2e_steps = max(2, min(args.steps, 5))
        e2e_step()
        barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(e2e_steps):
            e2e_step()
        a1.record()
        barrier()
        e2e_ms = a0.elapsed_time(a1)
        e2e_ms = max_over_ranks(e2e_ms, dist, "cuda")
        h2d = sum(x.numel() * x.element_size() for x in th.values() if x is not None)
        d2h = sum(x.numel() * x.element_size() for x in out)
        e2e = {"value": tokens_per_step * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    cpu = None
    parity = None
    if world == 1 and not args.no_cpu_baseline:
        v, threads, desc, secs = oracle_sample_tokens_per_s(w, inp, target_s=args.cpu_seconds)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc, "seconds": secs}
        parity = parity_report(mdn, w, inp, t, p, args, ws)

    others = None
    if world == 1 and args.config == 2 and not args.no_other_configs:
        others = {wl.CONFIGS[i].name: time_config(mdn, wl.CONFIGS[i], args.path, peaks) for i in (1, 3, 4)}

    ws_in = abytes
    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": n_warm, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": workload_desc(w), "path": mdn.resolved_path(p),
                   "parallelism": "independent batch per GPU, no collective",
                   "l2": ("inputs+outputs %.0f MB per step exceed the 126 MB L2; no flush between steps" % (ws_in / 1e6))
                         if n_copies == 1 else
                         ("inputs+outputs %.0f MB per step fit in the 126 MB L2: %d copies rotated (%.0f MB per round)"
                          % (ws_in / 1e6, n_copies, n_copies * ws_in / 1e6))},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline, "cpu_baseline": cpu, "parity": parity, "other_configs": others,
        "git": git_hash()}))
    if dist is not None:
        dist.destroy_process_group()


def run_decode(args):
    """Secondary benchmark (not the headline): mdn_decode_step, one token for each of `--decode-batch`
    sequences, H=16, dk=dv=128, bf16 tokens, fp32 states updated in place.  HBM-bound: every step reads
    and writes both dk x dv fp32 state matrices of every (sequence, head)."""
    import torch
    import paper_2605_05838_b200 as mdn
    mdn.lib()
    torch.cuda.set_device(0)
    B, H, d = args.decode_batch, 16, 128
    g = torch.Generator(device="cuda").manual_seed(0)
    mk = lambda *shape: torch.randn(*shape, device="cuda", generator=g)
    q = torch.nn.functional.normalize(mk(B, 1, H, d), dim=-1).to(torch.bfloat16)
    k = torch.nn.functional.normalize(mk(B, 1, H, d), dim=-1).to(torch.bfloat16)
    v = mk(B, 1, H, d).to(torch.bfloat16)
    beta = torch.full((B, 1, H), 0.03, device="cuda"); la = torch.full((B, 1, H), -0.08, device="cuda")
    lm = torch.full((B, 1, H), -0.03, device="cuda"); eta = torch.ones((B, 1, H), device="cuda")
    # several state sets so that consecutive steps do not find their state in the 126 MB L2
    n_sets = max(2, int(2 * L2_BYTES // (2 * B * H * d * d * 4)) + 1)
    states = [(0.02 * mk(B, H, d, d), 0.02 * mk(B, H, d, d)) for _ in range(n_sets)]
    o = torch.empty((B, 1, H, d), dtype=torch.bfloat16, device="cuda")

    ops = None
    if args.layer_ops:      # the same step with the layer's element-wise operations inside the kernel
        hv = lambda lo, hi: torch.rand(H, device="cuda", generator=g) * (hi - lo) + lo
        ops = mdn.make_layer_ops(q, v, gate_param=dict(a_alpha=hv(0.5, 8.0), b_alpha=hv(-4.5, -3.5), a_mu=hv(0.5, 8.0),
                                                       b_mu=hv(-3.5, -2.5), s=0.25, tau=11.3),
                                 qk_norm=dict(d=hv(-0.2, 0.5), eps=1e-6),
                                 out_norm_gate=dict(g=mk(B, 1, H, d).to(torch.bfloat16), w=None, eps=1e-5))

    def step(i):
        S, M = states[i % n_sets]
        mdn.decode_step(q, k, v, beta, la, lm, eta, S, M, out=o, layer_ops=ops)

    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    peaks = load_peaks()
    abytes = float(B * H * (4 * d * d * 4 + 3 * d * 2 + d * 2 + 16))
    print(json.dumps({
        "metric": "MDN decode step tokens/s", "value": B / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": "decode: B=%d,H=16,dk=dv=128, one token per sequence, fp32 states in place%s"
                               % (B, ", layer operations inside the kernel" if ops is not None else ""),
                   "l2": "%d rotating state sets (%.0f MB) exceed the 126 MB L2" % (n_sets, n_sets * 2 * B * H * d * d * 4 / 1e6)},
        "gpu_launches": args.steps,
        "roofline": {"bound": "hbm", "kernel": "decode_step", "achieved": abytes / (ms * 1e-3) / 1e9,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": abytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     # ncu dram bytes per launch at B=128 without the layer operations (profiles/decode_step_b128.md)
                     "traffic": 484.3e6 if (B == 128 and ops is None) else None,
                     "peak_source": peaks["source"], "algorithmic_bytes": abytes}}))


def run_layer_ops(args, w):
    """Secondary benchmark (not the headline): the forward with the layer's element-wise operations (gate
    parameterisation, q/k pre-processing, output norm + gate), once absorbed by the kernels and once as passes of
    their own around the unchanged forward.  Same workload, inputs resident in HBM, CUDA events."""
    import torch
    import paper_2605_05838_b200 as mdn
    mdn.lib()
    torch.cuda.set_device(0)
    inp = wl.make_layer_inputs(w)
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    dev = lambda x, d=torch.float32: torch.from_numpy(np.ascontiguousarray(x)).to("cuda").to(d)
    q, k, v, g = dev(inp["q"], dt), dev(inp["k"], dt), dev(inp["v"], dt), dev(inp["g"], dt)
    gates = [dev(inp[n]) for n in ("x_beta", "x_alpha", "x_mu", "x_eta")]
    gp = dict(a_alpha=dev(inp["a_alpha"]), b_alpha=dev(inp["b_alpha"]), a_mu=dev(inp["a_mu"]), b_mu=dev(inp["b_mu"]),
              s=inp["s"], tau=inp["tau"], log_mu_min=inp["log_mu_min"])
    dvec, wn = dev(inp["d"]), dev(inp["w_norm"])
    out = torch.empty_like(v)
    res = {}
    for mode in ("fused", "separate"):
        ops = mdn.make_layer_ops(q, v, gate_param=gp, qk_norm=dict(d=dvec, eps=inp["qk_eps"]),
                                 out_norm_gate=dict(g=g, w=wn, eps=inp["rms_eps"]), placement=mode)
        need = int(mdn.lib().mdn_chunk_fwd_fused_workspace_bytes(
            ctypes.byref(mdn.make_params(q, v, scale=inp["scale"], path=args.path)), ctypes.byref(ops)))
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")

        def step():
            mdn.chunk_fwd(q, k, v, *gates, scale=inp["scale"], path=args.path, layer_ops=ops, workspace=ws, out=out)

        for _ in range(max(args.warmup, 3)):
            step()
        launches = mdn.last_launch_count()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        res[mode] = {"ms_per_step": e0.elapsed_time(e1) / args.steps, "launches_per_step": launches}
    tokens = w.B * w.T
    peaks = load_peaks()
    es = 2 if w.dtype == "bf16" else 4
    # algorithmic bytes of the whole step: q, k, v, g read and o written once, four fp32 raw gates, final states
    abytes = float(tokens * w.H * ((2 * w.dk + 3 * w.dv) * es + 16) + 2 * w.B * w.H * w.dk * w.dv * 4)
    ach = abytes / (res["fused"]["ms_per_step"] * 1e-3) / 1e9
    print(json.dumps({
        "roofline": {"bound": "hbm", "kernel": "whole step (two kernels)", "achieved": ach, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                     "algorithmic_bytes": abytes},
        "metric": "MDN chunkwise fwd with layer ops tokens/s", "value": tokens / (res["fused"]["ms_per_step"] * 1e-3),
        "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": res["fused"]["ms_per_step"], "higher_is_better": True, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": workload_desc(w), "ops": "gate parameterisation + q/k L2Norm(q - d k) + RMSNorm*sigmoid gate"},
        "gpu_launches": res["fused"]["launches_per_step"] * args.steps,
        "placement": {"inside the kernels": res["fused"], "separate passes": res["separate"]}}))


def run_backward(args, w):
    """Secondary benchmark (not the headline): the backward (all gradients) on the same workload, inputs and the
    upstream gradient resident in HBM, CUDA events.  --bwd-method chunked (default where it applies: bf16, dk = dv = 128,
    fixed length): mdn_chunk_bwd_chunked, the chunk-parallel tensor-core backward; stepwise: mdn_chunk_bwd, the exact
    token-level one."""
    import torch
    import paper_2605_05838_b200 as mdn
    mdn.lib()
    torch.cuda.set_device(0)
    inp = wl.make_inputs(w)
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    dev = lambda x, d=torch.float32: None if x is None else torch.from_numpy(np.ascontiguousarray(x)).to("cuda").to(d)
    q, k, v = dev(inp["q"], dt), dev(inp["k"], dt), dev(inp["v"], dt)
    gates = [dev(inp[n]) for n in ("beta", "log_alpha", "log_mu", "eta")]
    cu = None if inp["cu_seqlens"] is None else torch.from_numpy(inp["cu_seqlens"]).to("cuda")
    d_o = torch.randn(v.shape, device="cuda", generator=torch.Generator(device="cuda").manual_seed(1)).to(dt)
    can_chunk = w.dtype == "bf16" and w.dk == 128 and w.dv == 128
    method = args.bwd_method if args.bwd_method != "auto" else ("chunked" if can_chunk else "stepwise")
    if method == "chunked":
        need = int(mdn.lib().mdn_chunk_bwd_chunked_workspace_bytes(ctypes.byref(
            mdn.make_params(q, v, num_seqs=0 if cu is None else cu.numel() - 1, path="tensor"))))
    else:
        need = int(mdn.lib().mdn_chunk_bwd_workspace_bytes(ctypes.byref(mdn.make_params(q, v, num_seqs=0 if cu is None else cu.numel() - 1))))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    S0, M0 = dev(inp["S0"]), dev(inp["M0"])

    def step():
        return mdn.chunk_bwd(q, k, v, *gates, d_o, initial_S=S0, initial_M=M0, cu_seqlens=cu,
                             scale=inp["scale"], workspace=ws, method=method)

    warm = max(args.warmup, 3)
    for _ in range(warm):
        step()
    launches = mdn.last_launch_count()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    train = None
    if method == "chunked":
        # the save-for-backward split: a forward that keeps its chunk states, then the backward on what it kept
        fkw = dict(initial_S=S0, initial_M=M0, cu_seqlens=cu, scale=inp["scale"], path="tensor")
        o_buf = torch.empty_like(v)

        def timed(fn, n):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record()
            for _ in range(n):
                fn()
            t1.record()
            torch.cuda.synchronize()
            return t0.elapsed_time(t1) / n

        _, _, _, states, fws = mdn.chunk_fwd(q, k, v, *gates, keep_chunk_states=True, out=o_buf, **fkw)
        f_ms = timed(lambda: mdn.chunk_fwd(q, k, v, *gates, keep_chunk_states=True, out=o_buf, workspace=fws, **fkw), args.steps)
        ws2 = torch.empty(int(mdn.lib().mdn_chunk_bwd_saved_workspace_bytes(ctypes.byref(
            mdn.make_params(q, v, num_seqs=0 if cu is None else cu.numel() - 1, path="tensor")))), dtype=torch.uint8, device="cuda")
        b_ms = timed(lambda: mdn.chunk_bwd(q, k, v, *gates, d_o, initial_S=S0, initial_M=M0, cu_seqlens=cu, scale=inp["scale"],
                                           workspace=ws2, method="chunked", saved=(fws, states)), args.steps)
        train = {"forward_keep_states_ms": f_ms, "backward_on_saved_states_ms": b_ms,
                 "tokens_per_s": w.B * w.T / ((f_ms + b_ms) * 1e-3)}
    peaks = load_peaks()
    tokens, es = w.B * w.T, (2 if w.dtype == "bf16" else 4)
    # reads q, k, v, dO and four gates; writes dq, dk, dv (fp32) and four gate gradients
    abytes = float(tokens * w.H * ((2 * w.dk + 2 * w.dv) * es + 16 + (2 * w.dk + w.dv) * 4 + 16))
    print(json.dumps({
        "metric": "MDN chunkwise bwd tokens/s", "value": tokens / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": args.steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True,
        "dtype": "bf16" if method == "chunked" else "f32",
        "data": "synthetic", "config": {"workload": workload_desc(w), "form": (
            "chunk-parallel: state-only forward keeping the chunk states, adjoint state chain, per-chunk kernel "
            "(bf16 tensor-core products, fp32 accumulation)" if method == "chunked" else
            "token-level adjoint recurrence, per-chunk checkpoints and recomputation (fp32)")},
        "gpu_launches": launches * args.steps, "workspace_bytes": need, "training_step": train,
        "roofline": {"bound": "hbm", "kernel": "whole backward" if method == "chunked" else "bwd_stepwise", "achieved": abytes / (ms * 1e-3) / 1e9,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": abytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "traffic": None, "peak_source": peaks["source"], "algorithmic_bytes": abytes}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=2, help="index into the named workloads (2 = headline)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the short timings of configs 1, 3 and 4")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--decode", action="store_true", help="secondary benchmark: the recurrent decode step")
    ap.add_argument("--decode-batch", type=int, default=128)
    ap.add_argument("--bwd-method", default="auto", choices=["auto", "chunked", "stepwise"])
    ap.add_argument("--backward", action="store_true", help="secondary benchmark: mdn_chunk_bwd (all gradients)")
    ap.add_argument("--layer-ops", action="store_true",
                    help="secondary benchmark: forward with the layer's element-wise operations, fused vs separate passes")
    args = ap.parse_args()
    if args.decode:
        run_decode(args)
        return
    w = wl.CONFIGS[args.config]
    if args.layer_ops and not args.decode:
        run_layer_ops(args, w)
        return
    if args.backward:
        run_backward(args, w)
        return
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
