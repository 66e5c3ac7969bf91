#!/usr/bin/env python
"""Device-time measurements of the workloads next to the headline one (bench.py times config 1).

    python bench_configs.py [--only mask,dynamic,...] [--seconds S] [--cfg4-batch B]

Each workload is one record: config 1 with the gate mask emitted, with time-varying retention, with
the Ear epilogue and with bf16 storage; config 2 (chunked prefill, 4096-token calls with the state
carried, issued call by call and replayed from a CUDA graph); config 3 (backward: reverse scan +
reductions, static and time-varying retention); config 4 (fused mixing path forward, and its
backward); single-token decode.  ``bench.py`` imports :func:`run_records` and puts the records of
the benchmark configs into its JSON line; run on its own, this file prints one JSON line per record
(the form the ncu captures under ``profiles/`` use, with ``--only`` and a small ``--seconds``).

How a record is timed: warm-up steps, then blocks of ``n`` steps, each block between two CUDA events
on the launching stream, issued back to back without a host synchronisation until about
``--seconds`` of device time have been queued; the record reports the median block (and the
fastest and slowest).  Steps rotate over several buffer sets larger than L2.  SM clocks and
throttle reasons come from one ``nvidia-smi`` process that samples every 20 ms for the whole run;
a record takes the samples whose timestamps fall inside its own timed window.

The large arrays are drawn on the device (torch generator, seeded) with the distributions of
``paper_2604_04250_b200.inputs``; parameters (retention, rotation, conv taps) come from that
module's numpy recipe.
"""
from __future__ import annotations

import argparse
import datetime
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np


# Kernel launches (and memsets) one call of the multi-launch entry points makes.
LAUNCHES = {"bwd": 2, "bwd_dynamic": 2, "mixing_bwd": 2, "mixing_bwd_dynamic": 2}


def measured_peak():
    """HBM copy bandwidth measured on this machine (GB/s), else the fallback figure."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """One nvidia-smi process sampling SM clock, power and throttle reasons every 20 ms, with
    timestamps; :meth:`window` summarises the samples between two host times."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.samples = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
        time.sleep(0.1)
        return self

    def stop(self):
        """Ends the sampling process and parses what it printed."""
        self.samples = []
        if self.proc is None:
            return
        time.sleep(0.1)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        self.proc = None
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                t = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.samples.append((t, float(f[1]), float(f[2]), float(f[3]),
                                     [n for n, v in zip(self.NAMES, f[4:8]) if v.lower().startswith("active")]))
            except ValueError:
                continue

    def window(self, t0, t1):
        """Clock summary of the samples taken between host times t0 and t1 (after :meth:`stop`)."""
        if self.samples is None:
            self.stop()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        sel = [s for s in self.samples if t0 <= s[0] <= t1]
        if not sel:                                  # a window shorter than the sampling period
            mid = 0.5 * (t0 + t1)
            sel = [min(self.samples, key=lambda s: abs(s[0] - mid))]
        reasons = sorted({r for s in sel for r in s[4]})
        return {"sm_mhz": statistics.median(s[1] for s in sel), "sm_max_mhz": max(s[2] for s in sel),
                "power_w": round(statistics.median(s[3] for s in sel), 1), "samples": len(sel), "reasons": reasons}


def timed_blocks(step, n, seconds=0.4, warmup=3, min_blocks=5, max_blocks=400, prewarm=0, stream=None):
    """Times blocks of ``n`` calls of ``step(i)``: after ``warmup`` + ``prewarm`` untimed steps the
    blocks are issued back to back, an event between one block and the next, no host
    synchronisation until all are queued.  Returns (per-block milliseconds, host window)."""
    import torch
    st = stream or torch.cuda.current_stream()
    k = 0
    for _ in range(warmup):
        step(k)
        k += 1
    torch.cuda.synchronize()
    # one measured block sizes the run
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st)
    for _ in range(n):
        step(k)
        k += 1
    e1.record(st)
    torch.cuda.synchronize()
    first = max(e0.elapsed_time(e1), 1e-3)
    blocks = int(min(max(min_blocks, math.ceil(seconds * 1e3 / first)), max_blocks))
    for _ in range(prewarm):                          # the timed blocks start on a busy, clocked-up GPU
        step(k)
        k += 1
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(blocks + 1)]
    t0 = time.time()
    evs[0].record(st)
    for b in range(blocks):
        for _ in range(n):
            step(k)
            k += 1
        evs[b + 1].record(st)
    torch.cuda.synchronize()
    t1 = time.time()
    return [evs[b].elapsed_time(evs[b + 1]) for b in range(blocks)], (t0, t1)


def record(name, tokens, nbytes, launches, times_ms, n, window, note=None, extra=None):
    """One workload's record; clocks are filled in later from the sampler."""
    peak, kind = measured_peak()
    ms = statistics.median(times_ms) / n
    gbs = nbytes / (ms * 1e-3) / 1e9
    r = {"workload": name, "ms": ms, "ms_min": min(times_ms) / n, "ms_max": max(times_ms) / n,
         "blocks": len(times_ms), "steps_per_block": n, "launches_per_step": launches,
         "Mtokens_per_s": tokens / (ms * 1e-3) / 1e6, "algorithmic_GBps": gbs,
         "frac": gbs / peak, "peak_kind": kind + " copy bandwidth", "frac_of_nominal_8000": gbs / 8000.0,
         "_window": window}
    if note:
        r["note"] = note
    if extra:
        r.update(extra)
    return r


def attach_clocks(records, sampler):
    for r in records:
        t0, t1 = r.pop("_window")
        c = sampler.window(t0, t1)
        r["clocks"] = c
        if c.get("sm_mhz"):
            r["us_x_sm_ghz"] = r["ms"] * 1e3 * c["sm_mhz"] / 1e3     # time x clock: compares power-capped runs
    return records


# ---- inputs on the device -------------------------------------------------------------------------
def _gen(seed):
    import torch
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return g


def dev_pushes(B, L, C, seed):
    """complex64 pushes, magnitude U[0,1), phase U[-pi,pi)."""
    import torch
    g = _gen(seed)
    m = torch.rand((B, L, C), generator=g, device="cuda")
    ph = (torch.rand((B, L, C), generator=g, device="cuda") * 2.0 - 1.0) * math.pi
    return torch.polar(m, ph)


def dev_normal(shape, seed, std=1.0):
    import torch
    return torch.randn(shape, generator=_gen(seed), device="cuda") * std


def dev_cnormal(shape, seed):
    import torch
    return torch.view_as_complex(torch.randn(tuple(shape) + (2,), generator=_gen(seed), device="cuda"))


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


# ---- the workloads ------------------------------------------------------------------------------
def cfg1_variants(cb, inputs, want, seconds):
    import torch
    out = []
    if not any(want(x) for x in ("plain", "mask", "ear", "bf16", "dynamic")):
        return out
    cfg = inputs.CONFIGS[1]
    B, L, C = cfg.B, cfg.L, cfg.C
    small = inputs.scan_inputs(1, 1, C, cfg.seed, cfg.gamma_lo, cfg.gamma_hi)
    g, t = _dev(small["gamma"]), _dev(small["theta"])
    NS = 6
    ps = [dev_pushes(B, L, C, cfg.seed + 10 * i) for i in range(NS)]
    ys = [torch.empty_like(ps[0]) for _ in range(NS)]
    IND = cb.CAWN_FLAG_INPUT_INDEPENDENT
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=IND)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    n = 20
    if want("plain"):
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd(prm, ps[i % NS], g, t, ys[i % NS], ws), n, seconds, prewarm=50)
        out.append(record("cfg1_train_fwd", B * L, B * L * C * 16, 1, tm, n, win))
    if want("mask"):
        masks = [torch.zeros((B, L, C // 32), dtype=torch.int32, device="cuda") for _ in range(NS)]
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd(prm, ps[i % NS], g, t, ys[i % NS], ws, gate_mask=masks[i % NS]),
                               n, seconds, prewarm=50)
        out.append(record("cfg1_train_fwd+mask", B * L, B * L * C * (16 + 0.125), 1, tm, n, win))
        del masks
    if want("ear"):
        ew, eb = dev_normal((2 * cfg.H, 3), 5), dev_normal((2 * cfg.H,), 6)
        zs = [y.view(torch.float32).view(B, L, 2, C) for y in ys]      # planar rows are as long as interleaved ones
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd_ear(prm, ps[i % NS], g, t, ew, 3, zs[i % NS], ws, ear_bias=eb),
                               n, seconds, prewarm=50)
        out.append(record("cfg1_train_fwd+ear_conv", B * L, B * L * C * 16, 1, tm, n, win))
    if want("bf16"):
        p16 = [p.view(torch.float32).to(torch.bfloat16).view(B, L, C, 2) for p in ps]
        y16 = [torch.empty((B, L, C, 2), dtype=torch.bfloat16, device="cuda") for _ in range(NS)]
        for name, fl, xin, yout, nbytes in (
                ("cfg1_train_fwd_bf16_in+out", cb.CAWN_FLAG_INPUT_BF16 | cb.CAWN_FLAG_OUTPUT_BF16, p16, y16, 8),
                ("cfg1_train_fwd_bf16_out", cb.CAWN_FLAG_OUTPUT_BF16, ps, y16, 12)):
            prm16 = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=IND | fl)
            tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd(prm16, xin[i % NS], g, t, yout[i % NS], ws),
                                   n, seconds, prewarm=50)
            out.append(record(name, B * L, B * L * C * nbytes, 1, tm, n, win))
        del p16, y16
    if want("dynamic"):
        dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
        gl, fb = _dev(dd["gamma_logit"]), _dev(dd["freq_bias"])
        prm_d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=IND | cb.CAWN_FLAG_RETENTION_DYNAMIC)
        ws_d = cb.new_workspace(prm_d, cb.CAWN_OP_FWD)
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd(prm_d, ps[i % NS], None, t, ys[i % NS], ws_d, gamma_logit=gl, freq_bias=fb),
                               n, seconds, prewarm=50)
        assert cb.cawn_poll_status(ws_d) == 0
        out.append(record("cfg1_train_fwd_dynamic_retention", B * L, B * L * (C * 16 + cfg.H * 4), 1, tm, n, win,
                          note="the paper's per-token, per-head retention"))
    assert cb.cawn_poll_status(ws) == 0
    return out


def cfg2_prefill(cb, inputs, want, seconds):
    import torch
    out = []
    if not want("cfg2"):
        return out
    cfg = inputs.CONFIGS[2]
    C, n = cfg.C, cfg.chunk
    small = inputs.scan_inputs(1, 1, C, cfg.seed, cfg.gamma_lo, cfg.gamma_hi)
    g, t = _dev(small["gamma"]), _dev(small["theta"])
    chunks = [dev_pushes(cfg.B, n, C, cfg.seed + 10 * i) for i in range(16)]     # 16 distinct chunks (805 MB), cycled
    ys = [torch.empty_like(chunks[0]) for _ in range(4)]
    state = torch.zeros((cfg.B, C), dtype=torch.complex64, device="cuda")
    prm = cb.make_params(cfg.B, n, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=cb.CAWN_FLAG_INPUT_INDEPENDENT)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    ncalls = 64

    def prefill(i):
        st = torch.cuda.current_stream().cuda_stream      # looked up once per 64 calls, not per call
        for j in range(ncalls):
            cb.cawn_phase_accumulate_fwd(prm, chunks[j % 16], g, t, ys[j % 4], ws, state_in=state, state_out=state, stream=st)
    if want("cfg2"):
        tm, win = timed_blocks(prefill, 1, seconds, warmup=2)
        assert cb.cawn_poll_status(ws) == 0
        r = record("cfg2_chunked_prefill", ncalls * n, ncalls * n * C * 16, ncalls, tm, 1, win,
                   note="64 calls of 4096 tokens per step, one launch per call, state carried on the device")
        r["us_per_4096_token_call"] = r["ms"] * 1e3 / ncalls
        out.append(r)
        # the same 64 calls recorded once into a CUDA graph: takes the host's per-call cost out
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            prefill(0)
        tm, win = timed_blocks(lambda i: graph.replay(), 1, seconds, warmup=2)
        assert cb.cawn_poll_status(ws) == 0
        r = record("cfg2_chunked_prefill_cuda_graph", ncalls * n, ncalls * n * C * 16, ncalls, tm, 1, win,
                   note="the same 64 calls replayed from one CUDA graph")
        r["us_per_4096_token_call"] = r["ms"] * 1e3 / ncalls
        out.append(r)
    return out


def cfg3_backward(cb, inputs, want, seconds):
    import torch
    out = []
    if not (want("cfg3") or want("cfg3dyn")):
        return out
    cfg = inputs.CONFIGS[3]
    B, L, C = cfg.B, cfg.L, cfg.C
    small = inputs.scan_inputs(1, 1, C, cfg.seed, cfg.gamma_lo, cfg.gamma_hi)
    g, t = _dev(small["gamma"]), _dev(small["theta"])
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps)
    NS = 3
    P = torch.empty((B, L, C), dtype=torch.complex64, device="cuda")
    wf = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    cb.cawn_phase_accumulate_fwd(prm, dev_pushes(B, L, C, cfg.seed), g, t, P, wf)
    Ps = [P.clone() for _ in range(NS)]
    gys = [dev_cnormal((B, L, C), cfg.seed + 20 + i) for i in range(NS)]
    gps = [torch.empty_like(P) for _ in range(NS)]
    gg, gt = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    gsi = torch.empty((B, C), dtype=torch.complex64, device="cuda")
    wb = cb.new_workspace(prm, cb.CAWN_OP_BWD_SAVED)
    n = 10
    if want("cfg3"):
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_bwd(prm, Ps[i % NS], cb.CAWN_SAVED_STATES, g, t, gys[i % NS], gps[i % NS],
                                                                      wb, grad_gamma=gg, grad_theta=gt, grad_state_in=gsi),
                               n, seconds, prewarm=20)
        assert cb.cawn_poll_status(wb) == 0
        out.append(record("cfg3_bwd", B * L, B * L * C * 24, LAUNCHES["bwd"], tm, n, win,
                          note="reads grad_y and the saved states, writes grad_p; reverse scan + the reduction of the parameter sums"))
    if want("cfg3dyn"):
        dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
        gl, fb = _dev(dd["gamma_logit"]), _dev(dd["freq_bias"])
        prm_d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
        ggl, gfb = torch.empty((B, L, cfg.H), device="cuda"), torch.empty(cfg.F, device="cuda")
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_bwd_dynamic(prm_d, Ps[i % NS], cb.CAWN_SAVED_STATES, gl, fb, t, gys[i % NS],
                                                                              gps[i % NS], wb, grad_gamma_logit=ggl, grad_freq_bias=gfb,
                                                                              grad_theta=gt, grad_state_in=gsi),
                               n, seconds, prewarm=20)
        assert cb.cawn_poll_status(wb) == 0
        out.append(record("cfg3_bwd_dynamic_retention", B * L, B * L * (C * 24 + cfg.H * 8), LAUNCHES['bwd_dynamic'], tm, n, win,
                          note="the paper's per-token retention: adds the logit and frequency-bias gradients"))
    return out


def cfg4_fused(cb, inputs, want, seconds, batch=0):
    import torch
    out = []
    if not any(want(x) for x in ("cfg4", "cfg4dyn", "cfg4bf16", "cfg4bwd", "cfg4bwddyn")):
        return out
    cfg = inputs.CONFIGS[4]
    B, L, C = (batch or cfg.B), cfg.L, cfg.C
    tag = "" if B == cfg.B else "_B%d" % B
    small = inputs.fused_inputs(1, 1, C, cfg.seed, cfg.conv_k, cfg.gamma_lo, cfg.gamma_hi)
    g, t, w = _dev(small["gamma"]), _dev(small["theta"]), _dev(small["conv_w"])
    tau = float(inputs.gate_tau(cfg.gate_eps))
    IND = cb.CAWN_FLAG_INPUT_INDEPENDENT
    NS = 2
    hs = [dev_normal((B, L, C), cfg.seed + 10 * i) for i in range(NS)]
    ys = [torch.empty((B, L, C), dtype=torch.complex64, device="cuda") for _ in range(NS)]
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=tau, conv_k=cfg.conv_k, flags=IND)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    n = 4
    if want("cfg4"):
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd(prm, hs[i % NS], g, t, ys[i % NS], ws, conv_w=w), n, seconds, prewarm=8)
        assert cb.cawn_poll_status(ws) == 0
        out.append(record("cfg4_fused" + tag, B * L, B * L * C * 12, 1, tm, n, win,
                          note="conv prelude, phasor map, gate, push and scan in one kernel: reads h (4 B), writes y (8 B) per element"))
    if want("cfg4dyn"):
        dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
        gl, fb = _dev(dd["gamma_logit"]), _dev(dd["freq_bias"])
        prm_d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=tau, conv_k=cfg.conv_k,
                               flags=IND | cb.CAWN_FLAG_RETENTION_DYNAMIC)
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd(prm_d, hs[i % NS], None, t, ys[i % NS], ws, conv_w=w,
                                                                      gamma_logit=gl, freq_bias=fb), n, seconds, prewarm=8)
        assert cb.cawn_poll_status(ws) == 0
        out.append(record("cfg4_fused_dynamic_retention" + tag, B * L, B * L * (C * 12 + cfg.H * 4), 1, tm, n, win))
        ew, eb = dev_normal((2 * cfg.H, 3), 5), dev_normal((2 * cfg.H,), 6)
        zs = [y.view(torch.float32).view(B, L, 2, C) for y in ys]
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd_ear(prm_d, hs[i % NS], None, t, ew, 3, zs[i % NS], ws, ear_bias=eb,
                                                                          conv_w=w, gamma_logit=gl, freq_bias=fb), n, seconds, prewarm=8)
        assert cb.cawn_poll_status(ws) == 0
        out.append(record("cfg4_fused_dynamic_retention+ear_conv" + tag, B * L, B * L * (C * 12 + cfg.H * 4), 1, tm, n, win,
                          note="the paper's whole mixing step up to the Ear's convolution in one kernel"))
    if want("cfg4bf16"):
        prm16 = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=tau, conv_k=cfg.conv_k,
                               flags=IND | cb.CAWN_FLAG_INPUT_BF16 | cb.CAWN_FLAG_OUTPUT_BF16)
        h16 = [h.to(torch.bfloat16) for h in hs]
        y16 = [torch.empty((B, L, C, 2), dtype=torch.bfloat16, device="cuda") for _ in range(NS)]
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd(prm16, h16[i % NS], g, t, y16[i % NS], ws, conv_w=w), n, seconds, prewarm=8)
        assert cb.cawn_poll_status(ws) == 0
        out.append(record("cfg4_fused_bf16_in+out" + tag, B * L, B * L * C * 6, 1, tm, n, win))
        del h16, y16
        # the paper's own layer form: bf16 network around the fp32 scan, per-token retention, Ear conv
        dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
        gl, fb = _dev(dd["gamma_logit"]), _dev(dd["freq_bias"])
        prm16d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=tau, conv_k=cfg.conv_k,
                                flags=IND | cb.CAWN_FLAG_RETENTION_DYNAMIC | cb.CAWN_FLAG_INPUT_BF16 | cb.CAWN_FLAG_OUTPUT_BF16)
        ew, eb = dev_normal((2 * cfg.H, 3), 5), dev_normal((2 * cfg.H,), 6)
        h16 = [h.to(torch.bfloat16) for h in hs]
        z16 = [torch.empty((B, L, 2, C), dtype=torch.bfloat16, device="cuda") for _ in range(NS)]
        tm, win = timed_blocks(lambda i: cb.cawn_phase_accumulate_fwd_ear(prm16d, h16[i % NS], None, t, ew, 3, z16[i % NS], ws, ear_bias=eb,
                                                                          conv_w=w, gamma_logit=gl, freq_bias=fb), n, seconds, prewarm=8)
        assert cb.cawn_poll_status(ws) == 0
        out.append(record("cfg4_fused_dynamic_retention+ear_conv_bf16_in+out" + tag, B * L, B * L * (C * 6 + cfg.H * 4), 1, tm, n, win,
                          note="the paper's layer form: bf16 hidden states in, bf16 planar Z out, fp32 scan, per-token retention"))
        del h16, z16
    if want("cfg4bwd") or want("cfg4bwddyn"):
        h, P = hs[0], ys[0]
        prm_b = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=tau, conv_k=cfg.conv_k)
        cb.cawn_phase_accumulate_fwd(prm_b, h, g, t, P, ws, conv_w=w)
        gy = dev_cnormal((B, L, C), cfg.seed + 30)
        gh = hs[1]                                                # overwritten: no longer needed as an input
        gw, gb = torch.empty((C, cfg.conv_k), device="cuda"), torch.empty(C, device="cuda")
        gg, gt = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
        wb = cb.new_workspace(prm_b, cb.CAWN_OP_MIXING_BWD)
        if want("cfg4bwd"):
            tm, win = timed_blocks(lambda i: cb.cawn_mixing_bwd(prm_b, h, w, g, t, gy, gh, wb, saved_states=P, grad_conv_w=gw,
                                                                grad_conv_bias=gb, grad_gamma=gg, grad_theta=gt), 2, seconds, prewarm=4)
            assert cb.cawn_poll_status(wb) == 0
            out.append(record("cfg4_mixing_bwd" + tag, B * L, B * L * C * 24, LAUNCHES['mixing_bwd'], tm, 2, win,
                              note="reads grad_y (8 B), saved states (8 B), h (4 B), writes grad_h (4 B) per element; "
                                   "reverse scan with the prelude's chain rule and the conv transpose as its epilogue"))
        if want("cfg4bwddyn"):
            dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
            gl, fb = _dev(dd["gamma_logit"]), _dev(dd["freq_bias"])
            prm_d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=tau, conv_k=cfg.conv_k,
                                   flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
            cb.cawn_phase_accumulate_fwd(prm_d, h, None, t, P, ws, conv_w=w, gamma_logit=gl, freq_bias=fb)
            ggl, gfb = torch.empty((B, L, cfg.H), device="cuda"), torch.empty(cfg.F, device="cuda")
            tm, win = timed_blocks(lambda i: cb.cawn_mixing_bwd_dynamic(prm_d, h, w, gl, fb, t, gy, gh, wb, saved_states=P, grad_conv_w=gw,
                                                                        grad_conv_bias=gb, grad_gamma_logit=ggl, grad_freq_bias=gfb,
                                                                        grad_theta=gt), 2, seconds, prewarm=4)
            assert cb.cawn_poll_status(wb) == 0
            out.append(record("cfg4_mixing_bwd_dynamic_retention" + tag, B * L, B * L * (C * 24 + cfg.H * 8),
                              LAUNCHES['mixing_bwd_dynamic'], tm, 2, win))
    return out


def decode(cb, inputs, want, seconds):
    import torch
    out = []
    if not want("decode"):
        return out
    cfg = inputs.CONFIGS[4]
    B, C, n = 1, cfg.C, 256
    small = inputs.fused_inputs(1, 1, C, cfg.seed, cfg.conv_k, cfg.gamma_lo, cfg.gamma_hi)
    g, t, w = _dev(small["gamma"]), _dev(small["theta"]), _dev(small["conv_w"])
    prm = cb.make_params(B, 1, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=float(inputs.gate_tau(cfg.gate_eps)),
                         conv_k=cfg.conv_k)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    blob = torch.zeros(cb.cawn_workspace_bytes(prm, cb.CAWN_OP_STATE), dtype=torch.uint8, device="cuda")
    h = dev_normal((B, n, C), cfg.seed)
    rows = [h[:, i:i + 1].contiguous() for i in range(n)]
    y = torch.empty((B, 1, C), dtype=torch.complex64, device="cuda")

    def gen(i):
        for j in range(n):
            cb.cawn_phase_accumulate_fwd(prm, rows[j], g, t, y, ws, conv_w=w, state_in=blob, state_out=blob)
    tm, win = timed_blocks(gen, 1, seconds, warmup=2)
    assert cb.cawn_poll_status(ws) == 0
    r = record("decode_fused_B1_L1", n, n * C * 12, n, tm, 1, win,
               note="one launch per token from Python; latency-bound, bandwidth figures are not meaningful")
    r["us_per_token"] = r["ms"] * 1e3 / n
    out.append(r)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        gen(0)
    tm, win = timed_blocks(lambda i: graph.replay(), 1, seconds, warmup=2)
    assert cb.cawn_poll_status(ws) == 0
    r = record("decode_fused_B1_L1_cuda_graph", n, n * C * 12, n, tm, 1, win, note="256 decode steps replayed from one CUDA graph")
    r["us_per_token"] = r["ms"] * 1e3 / n
    out.append(r)
    return out


# The records bench.py puts into its line (the benchmark configs); everything else only on request.
DEFAULT = ("mask", "dynamic", "cfg2", "cfg3", "cfg3dyn", "cfg4", "cfg4bwd")
ALL = ("plain", "mask", "ear", "bf16", "dynamic", "cfg2", "cfg3", "cfg3dyn", "cfg4", "cfg4dyn", "cfg4bf16",
       "cfg4bwd", "cfg4bwddyn", "decode")


def run_records(only=DEFAULT, seconds=0.4, cfg4_batch=0):
    """Runs the selected workloads on the current device; records still carry their host windows
    (``_window``) for :func:`attach_clocks`."""
    import torch
    from paper_2604_04250_b200 import binding as cb, inputs
    cb.lib()
    only = set(only)
    want = lambda name: name in only
    out = []
    for fn in (cfg1_variants, cfg2_prefill, cfg3_backward):
        out += fn(cb, inputs, want, seconds)
        torch.cuda.empty_cache()
    out += cfg4_fused(cb, inputs, want, seconds, cfg4_batch)
    torch.cuda.empty_cache()
    out += decode(cb, inputs, want, seconds)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--only", default="", help="comma-separated subset of: " + ",".join(ALL) + " (default: all)")
    ap.add_argument("--seconds", type=float, default=0.4, help="device time queued per record")
    ap.add_argument("--cfg4-batch", type=int, default=0, help="batch rows of the config-4 records (0: the config's 16)")
    args = ap.parse_args()
    import torch
    torch.cuda.set_device(0)
    only = [x for x in args.only.split(",") if x] or list(ALL)
    sampler = ClockSampler(0).start()
    recs = run_records(only, args.seconds, args.cfg4_batch)
    sampler.stop()
    for r in attach_clocks(recs, sampler):
        print(json.dumps(r), flush=True)


if __name__ == "__main__":
    sys.exit(main())
