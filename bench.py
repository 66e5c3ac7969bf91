#!/usr/bin/env python
"""Benchmark of the phase-accumulation forward scan at d=768 (training shape).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one call of ``cawn_phase_accumulate_fwd`` (gate, chunk scan, inter-tile carry,
state out: one kernel launch) on B=8, L=2048, H=12 x F=64 complex64 pushes.  Steps rotate over
several independent buffer sets so that no step finds its inputs in L2.

Timing: W warm-up steps, then a stretch of untimed steps that brings the GPU to its clocks under
this load, then the block of K steps timed R times back to back (CUDA events on the launching
stream between the blocks, no host synchronisation in between); ``ms_per_step`` is the MEDIAN
block divided by K, the fastest and slowest blocks are reported beside it, and so is the time of
one launch alone (events around a single launch, the device idle before it).  SM clocks and
throttle reasons are sampled with ``nvidia-smi`` while the blocks run.

Prints ONE JSON line.  At one GPU the line also carries ``configs``: device-timed records of the
other benchmark configs (gate mask on, time-varying retention, chunked prefill, backward, the
fused mixing path and its backward), each with its own clock samples (``bench_configs.py``).
With ``--impl reference`` the fp64 CPU oracle is timed instead (on the host cores).
"""
from __future__ import annotations

import argparse
import hashlib
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

from bench_configs import ClockSampler, attach_clocks, measured_peak, run_records, DEFAULT as DEFAULT_RECORDS

METRIC = "phase_accumulation_fwd_scan_throughput_d768"
UNIT = "Mtokens/s"
NSETS = 6                      # rotating buffer sets: 6 x 201 MB = 1.2 GB >> 126 MB of L2
BYTES_PER_ELEMENT = 16         # algorithmic: read one complex64 push, write one complex64 output
REPEATS = 15                   # timed blocks of K steps; the median one is reported
PREWARM_S = 0.05               # untimed steps right before the timed blocks, in seconds of device time
# DRAM traffic of one launch of the headline kernel, read off an ncu capture: kept with the hash of
# the kernel sources it was taken from, and reported only while the sources still hash to that.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "cawn_scan_fwd_cfg1_traffic.json")


def workload():
    from paper_2604_04250_b200 import inputs
    return inputs.CONFIGS[1]


def csrc_hash():
    """sha256 over the kernel sources and the public header (names and contents, sorted)."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2604_04250_b200", "csrc")
    files = [os.path.join(csrc, f) for f in sorted(os.listdir(csrc))] + [os.path.join(ROOT, "include", "cawn.h")]
    for path in files:
        h.update(os.path.basename(path).encode())
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch, or None when the kernel has
    changed since the counters were taken (or none were)."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f)
        if rec.get("csrc_hash") == csrc_hash():
            return int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])
    except Exception:
        pass
    return None


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_worker(row, t_start, seconds):
    """One process of the all-core oracle timing: whole passes over one batch row of the workload
    (its own seeded row), counted inside the common window [t_start, t_start + seconds]."""
    import oracle
    from paper_2604_04250_b200 import inputs
    cfg = workload()
    d = inputs.scan_inputs(1, cfg.L, cfg.C, cfg.seed + 1 + row, cfg.gamma_lo, cfg.gamma_hi)
    oracle.forward(d["p"][:, :64], d["gamma"], d["theta"], cfg.gate_eps)        # load the library
    while time.time() < t_start:
        time.sleep(0.001)
    passes = 0
    while time.time() < t_start + seconds:
        oracle.forward(d["p"], d["gamma"], d["theta"], cfg.gate_eps)
        passes += 1
    print(json.dumps({"passes": passes, "elapsed": time.time() - t_start}))


def cpu_oracle_all_cores(cfg, seconds=6.0):
    """The unchanged oracle in one process per host core, each over its own batch row."""
    n = host_cores()
    t_start = time.time() + 4.0 + 0.02 * n                # every worker is loaded and waiting by then
    procs = [subprocess.Popen([sys.executable, os.path.abspath(__file__), "--oracle-worker", str(i), repr(t_start), str(seconds)],
                              stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, cwd=ROOT) for i in range(n)]
    passes, elapsed = 0, 0.0
    for p in procs:
        try:
            out, _ = p.communicate(timeout=seconds + 60)
            r = json.loads(out.strip().splitlines()[-1])
            passes += r["passes"]
            elapsed = max(elapsed, r["elapsed"])
        except Exception:
            p.kill()
    if passes == 0 or elapsed <= 0:
        return None
    return {"value": passes * cfg.L / elapsed / 1e6, "unit": UNIT, "processes": n,
            "sample": "%d passes over single batch rows (B=1, L=%d, C=%d) by %d processes in a %.1f s window"
                      % (passes, cfg.L, cfg.C, n, elapsed)}


def cpu_oracle_throughput(cfg, budget_s=8.0, min_passes=1):
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
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "host_cores": host_cores(), "kind": "oracle", "sample": sample},
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


def median_block(block_ms_per_rank_max):
    """The reported block: the median of the R per-block times (each already the max over ranks)."""
    return statistics.median(block_ms_per_rank_max)


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
    K = args.steps
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
    # one launch alone: the device idle before it, events right around it
    iso = []
    for i in range(12):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        step(i)
        b.record(stream)
        torch.cuda.synchronize()
        iso.append(a.elapsed_time(b))
    isolated_ms = statistics.median(iso)
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # Untimed steps first, so that the timed blocks start on a GPU that is busy and at its clocks
    # under this load; then R blocks of exactly K steps, an event between one block and the next
    # (an event between two launches makes the second wait for the first to drain, which back-to-back
    # calls on a stream do not do: hence one event per block, not per step).
    nwarm = max(50, int(PREWARM_S / (isolated_ms * 1e-3)))
    for i in range(nwarm):
        step(i)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(REPEATS + 1)]
    t0 = time.time()
    evs[0].record(stream)
    n = 0
    for r in range(REPEATS):
        for _ in range(K):
            step(args.warmup + n)
            n += 1
        evs[r + 1].record(stream)
    barrier()
    t1 = time.time()
    blocks = [evs[r].elapsed_time(evs[r + 1]) for r in range(REPEATS)]
    # the timed region lasts milliseconds and nvidia-smi samples every 20 ms: the same steps go on
    # (untimed) for half a second so that the samples describe the GPU under this very load
    t_load = time.perf_counter()
    while time.perf_counter() - t_load < 0.5:
        for i in range(50):
            step(i)
        torch.cuda.synchronize()
    t2 = time.time()
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
    e2e_steps = max(3, min(K, 10))
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
    del scratch, hp, hy, ps, ys, p0
    torch.cuda.empty_cache()

    red = reduce_max(blocks + [e2e_ms, isolated_ms], world, "cuda")
    blocks, e2e_ms, isolated_ms = red[:REPEATS], red[REPEATS], red[REPEATS + 1]
    total_ms = median_block(blocks)
    ms_per_step = total_ms / K

    # the other benchmark configs, one GPU only (they would hold N GPUs for a minute otherwise)
    records = []
    if world == 1 and not args.no_configs:
        records = run_records(DEFAULT_RECORDS, seconds=args.config_seconds)
    if rank == 0:
        sampler.stop()
        clocks_now = sampler.window(t0, t2)
        clocks_now["sm_mhz_timed_blocks"] = sampler.window(t0, t1).get("sm_mhz")
        attach_clocks(records, sampler)
    if rank == 0:
        peak, peak_kind = measured_peak()
        kernel_ms = ms_per_step                      # one kernel launch per step, back to back
        achieved = nelem * BYTES_PER_ELEMENT / (kernel_ms * 1e-3) / 1e9
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            v, passes, dt = cpu_oracle_throughput(cfg)
            cpu = {"value": v, "unit": UNIT, "cores": 1, "host_cores": host_cores(), "kind": "oracle",
                   "sample": "%d full passes of the same workload (B=%d L=%d C=%d) in %.1f s, one thread"
                             % (passes, B, L, C, dt),
                   "all_cores": cpu_oracle_all_cores(cfg)}
        line = {
            "metric": METRIC, "value": whole_job_value(world, tokens, ms_per_step), "unit": UNIT,
            "n_gpus": world, "steps": K, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": cfg.name, "B": B, "L": L, "H": cfg.H, "F": cfg.F,
                       "gate_eps": cfg.gate_eps, "per_gpu_tokens_per_step": tokens,
                       "l2": "steps rotate over %d buffer sets (%.2f GB) > 126 MB L2"
                             % (NSETS, NSETS * nelem * 16 / 1e9),
                       "parallelism": "independent batches per GPU, no collective"},
            "timing": {"blocks": REPEATS, "steps_per_block": K, "reported": "median block",
                       "ms_per_step_min": min(blocks) / K, "ms_per_step_max": max(blocks) / K,
                       "untimed_steps_before": nwarm, "isolated_launch_ms": isolated_ms,
                       "us_x_sm_ghz": (ms_per_step * clocks_now["sm_mhz"] if clocks_now.get("sm_mhz") else None)},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": peak_kind + " copy bandwidth",
                         "frac_of_nominal_8000": achieved / 8000.0,
                         "kernel": "cawn_scan_kernel<16,8,KIND_FWD,VEC,3> (no mask output)", "kernel_ms": kernel_ms,
                         "algorithmic_bytes_per_launch": nelem * BYTES_PER_ELEMENT,
                         "traffic": ncu_traffic()},
            "e2e": {"value": whole_job_value(world, tokens, e2e_ms), "unit": UNIT,
                    "h2d_bytes_per_step": nelem * 8 + 2 * C * 4, "d2h_bytes_per_step": nelem * 8 + B * C * 8,
                    "ms_per_step": e2e_ms, "api": "cawn_phase_accumulate_fwd_host (pinned host buffers)"},
            "gpu_launches": K,
            "clocks": clocks_now,
            "cpu_baseline": cpu,
            "configs": {r["workload"]: {k: v for k, v in r.items() if k != "workload"} for r in records},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    if len(sys.argv) > 1 and sys.argv[1] == "--oracle-worker":
        oracle_worker(int(sys.argv[2]), float(sys.argv[3]), float(sys.argv[4]))
        return
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the records of the other configs")
    ap.add_argument("--config-seconds", type=float, default=0.4, help="device time queued per config record")
    ap.add_argument("--print-csrc-hash", action="store_true", help="print the hash profiles/*_traffic.json is keyed on")
    args = ap.parse_args()
    if args.print_csrc_hash:
        print(csrc_hash())
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
