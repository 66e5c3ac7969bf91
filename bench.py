#!/usr/bin/env python
"""Benchmark of the phase-accumulation forward scan at d=768 (training shape).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one call of ``cawn_phase_accumulate_fwd`` (gate, chunk scan, inter-tile carry,
state out: one kernel launch) on B=8, L=2048, H=12 x F=64 complex64 pushes.  Steps rotate over
several independent buffer sets so that no step finds its inputs in L2.  Prints ONE JSON line.
With ``--impl reference`` the fp64 CPU oracle is timed instead (on the host cores).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "phase_accumulation_fwd_scan_throughput_d768"
UNIT = "Mtokens/s"
NSETS = 6                      # rotating buffer sets: 6 x 201 MB = 1.2 GB >> 126 MB of L2
BYTES_PER_ELEMENT = 16         # algorithmic: read one complex64 push, write one complex64 output
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the scan kernel on this
# workload, from the ncu capture summarised in profiles/cawn_scan_fwd_cfg1_ncu.md: 101.4 MB read
# + 47.4 MB written while an isolated launch runs (the rest of its 100.7 MB of output is still
# dirty in L2 when it ends).  Set to None whenever the kernel changes after the capture.
NCU_DRAM_BYTES_PER_LAUNCH = 151096576


def workload():
    from paper_2604_04250_b200 import inputs
    return inputs.CONFIGS[1]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def cpu_oracle_throughput(cfg, budget_s=10.0, min_passes=1):
    """Times the oracle (as it stands, one thread) on whole passes of the workload."""
    import oracle
    from paper_2604_04250_b200 import inputs
    d = inputs.config_inputs(cfg)
    oracle.forward(d["p"][:1, :64], d["gamma"], d["theta"], cfg.gate_eps)      # load the library
    passes, t0 = 0, time.perf_counter()
    while True:
        oracle.forward(d["p"], d["gamma"], d["theta"], cfg.gate_eps)
        passes += 1
        dt = time.perf_counter() - t0
        if passes >= min_passes and dt >= budget_s:
            break
    return cfg.B * cfg.L * passes / dt / 1e6, passes, dt


def run_reference(args):
    """The reference arm of this benchmark is the CPU oracle, timed on the host cores.

    Each step is a bounded sample of the workload: one batch row (B=1) of the same L and C.
    """
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2604_04250_b200 import inputs
    cfg = workload()
    d = inputs.config_inputs(cfg)
    oracle.build()
    row = d["p"][:1]
    for _ in range(max(args.warmup, 1)):
        oracle.forward(row[:, :256], d["gamma"], d["theta"], cfg.gate_eps)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.forward(row, d["gamma"], d["theta"], cfg.gate_eps)
    dt = time.perf_counter() - t0
    value = cfg.L * args.steps / dt / 1e6
    sample = "each step = one batch row (B=1, L=%d, C=%d) of the workload; fp64, sequential, 1 thread" % (cfg.L, cfg.C)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": cfg.name, "B": cfg.B, "L": cfg.L, "H": cfg.H, "F": cfg.F},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def rank_seed(cfg_seed, rank):
    """Every rank draws its own batch shard: same recipe, rank-specific seed."""
    return cfg_seed + 1000 * rank


def reduce_max(values, world, device):
    """Max over ranks of a few per-rank timings (the slowest rank defines the step time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_value(world, tokens_per_rank, ms_per_step):
    """Mtokens/s of all ranks together (weak scaling: every rank processes its own batch shard)."""
    return world * tokens_per_rank / (ms_per_step * 1e-3) / 1e6


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2604_04250_b200 import binding as cb, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    # a fresh checkout has no built library yet: the first local rank builds it (a no-op when it is
    # up to date), the others wait for it
    if local == 0:
        from paper_2604_04250_b200 import build as cuda_build
        cuda_build.build()
    if world > 1:
        dist.barrier()
    cb.lib()                                   # fails loudly if the CUDA library is still missing

    cfg = workload()
    B, L, C = cfg.B, cfg.L, cfg.C
    tokens = B * L
    nelem = tokens * C
    # every step reads a buffer set that no earlier step writes: the calls may overlap their tails
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=cb.CAWN_FLAG_INPUT_INDEPENDENT)
    d = inputs.scan_inputs(B, L, C, rank_seed(cfg.seed, rank), cfg.gamma_lo, cfg.gamma_hi)
    gamma = torch.from_numpy(d["gamma"]).cuda()
    theta = torch.from_numpy(d["theta"]).cuda()
    p0 = torch.from_numpy(d["p"]).cuda()
    # independent buffer sets (same values, rolled along time so no two sets are identical)
    ps = [torch.roll(p0, shifts=17 * i, dims=1).contiguous() for i in range(NSETS)]
    ys = [torch.empty_like(p0) for _ in range(NSETS)]
    state = torch.empty((B, C), dtype=torch.complex64, device="cuda")
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    stream = torch.cuda.current_stream()

    def step(i):
        s = i % NSETS
        cb.cawn_phase_accumulate_fwd(prm, ps[s], gamma, theta, ys[s], ws, state_out=state, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    # The timed region lasts a few milliseconds, nvidia-smi samples every 20 ms: the clocks are
    # sampled over the K timed steps plus the same steps repeated (untimed) for about half a second
    # right after them, so that the samples describe the GPU under this very load.
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.05)
    # two events bracket the K steps: an event between two launches would make each launch wait for
    # the one before to drain completely, which back-to-back calls on a stream do not do
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for i in range(args.steps):
        step(args.warmup + i)
    ev1.record(stream)
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    t_load = time.perf_counter()
    while time.perf_counter() - t_load < 0.5:
        for i in range(50):
            step(i)
        torch.cuda.synchronize()
    clocks_now = sampler.stop() if rank == 0 else None
    status = cb.cawn_poll_status(ws)
    if status != 0:
        raise RuntimeError("device status: " + cb.status_string(status))

    # end to end through the host-buffer entry point (pinned host memory, copies timed)
    scratch = cb.new_workspace(prm, cb.CAWN_OP_FWD_HOST)
    hp = torch.from_numpy(d["p"]).pin_memory()
    hg = torch.from_numpy(d["gamma"]).pin_memory()
    ht = torch.from_numpy(d["theta"]).pin_memory()
    hy = torch.empty((B, L, C), dtype=torch.complex64).pin_memory()
    hs = torch.empty((B, C), dtype=torch.complex64).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        cb.cawn_phase_accumulate_fwd_host(prm, hp, hg, ht, hy, scratch, state_out_host=hs, stream=stream)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        cb.cawn_phase_accumulate_fwd_host(prm, hp, hg, ht, hy, scratch, state_out_host=hs, stream=stream)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps

    total_ms, e2e_ms = reduce_max([total_ms, e2e_ms], world, "cuda")
    ms_per_step = total_ms / args.steps

    if rank == 0:
        peak, peak_kind = measured_peak()
        kernel_ms = ms_per_step                      # one kernel launch per step, back to back
        achieved = nelem * BYTES_PER_ELEMENT / (kernel_ms * 1e-3) / 1e9
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            v, passes, dt = cpu_oracle_throughput(cfg)
            cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                   "sample": "%d full passes of the same workload (B=%d L=%d C=%d) in %.1f s, one thread"
                             % (passes, B, L, C, dt)}
        line = {
            "metric": METRIC, "value": whole_job_value(world, tokens, ms_per_step), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": cfg.name, "B": B, "L": L, "H": cfg.H, "F": cfg.F,
                       "gate_eps": cfg.gate_eps, "per_gpu_tokens_per_step": tokens,
                       "l2": "steps rotate over %d buffer sets (%.2f GB) > 126 MB L2"
                             % (NSETS, NSETS * nelem * 16 / 1e9),
                       "parallelism": "independent batches per GPU, no collective"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": peak_kind + " copy bandwidth",
                         "frac_of_nominal_8000": achieved / 8000.0,
                         "kernel": "cawn_scan_kernel<16,8,KIND_FWD,VEC,3> (no mask output)", "kernel_ms": kernel_ms,
                         "algorithmic_bytes_per_launch": nelem * BYTES_PER_ELEMENT,
                         "traffic": NCU_DRAM_BYTES_PER_LAUNCH},
            "e2e": {"value": whole_job_value(world, tokens, e2e_ms), "unit": UNIT,
                    "h2d_bytes_per_step": nelem * 8 + 2 * C * 4, "d2h_bytes_per_step": nelem * 8 + B * C * 8,
                    "ms_per_step": e2e_ms, "api": "cawn_phase_accumulate_fwd_host (pinned host buffers)"},
            "gpu_launches": args.steps,
            "clocks": clocks_now,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
