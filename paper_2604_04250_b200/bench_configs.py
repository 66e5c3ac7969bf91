"""Device-time measurements of the other benchmark configs (bench.py times config 1 only).

    python -m paper_2604_04250_b200.bench_configs [--steps K] [--warmup W]

Prints one JSON line per workload: config 3 (backward, saved states), config 4 (fused mixing
path), config 2 (chunked prefill, a window of 4096-token calls with state passing), config 1 with
the mask emitted, and config 1 with time-varying retention.  Inputs are the seeded synthetic
arrays of ``inputs.py``, resident on the device; steps rotate over several buffer sets so that
no step finds its inputs in L2; K steps are timed between two CUDA events.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np


def _peak():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    try:
        with open(os.path.join(root, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def _time(step, steps, warmup):
    import torch
    st = torch.cuda.current_stream()
    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st)
    for i in range(steps):
        step(warmup + i)
    e1.record(st)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def _report(name, tokens, bytes_per_step, ms, launches, extra=None):
    peak, kind = _peak()
    gbs = bytes_per_step / (ms * 1e-3) / 1e9
    line = {"workload": name, "ms_per_step": ms, "Mtokens_per_s": tokens / (ms * 1e-3) / 1e6,
            "algorithmic_GBps": gbs, "frac_of_%s_copy_peak" % kind: gbs / peak,
            "frac_of_nominal_8000": gbs / 8000.0, "launches_per_step": launches}
    if extra:
        line.update(extra)
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--only", default="", help="comma-separated subset of: mask,ear,bf16,dynamic,cfg3,cfg4,cfg4bwd,cfg2,decode")
    ap.add_argument("--cfg4-batch", type=int, default=0, help="batch rows of the config-4 run (0: the config's 16)")
    args = ap.parse_args()
    only = set(x for x in args.only.split(",") if x)
    want = lambda name: not only or name in only
    import torch
    from . import binding as cb, inputs
    cb.lib()
    torch.cuda.set_device(0)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    IND = cb.CAWN_FLAG_INPUT_INDEPENDENT

    # ---- config 1 with the gate mask emitted, and with time-varying retention -----------------
    cfg = inputs.CONFIGS[1]
    B, L, C = cfg.B, cfg.L, cfg.C
    d = inputs.scan_inputs(B, L, C, cfg.seed, cfg.gamma_lo, cfg.gamma_hi)
    g, t, p0 = dev(d["gamma"]), dev(d["theta"]), dev(d["p"])
    NS = 6
    ps = [torch.roll(p0, 17 * i, 1).contiguous() for i in range(NS)]
    ys = [torch.empty_like(p0) for _ in range(NS)]
    masks = [torch.zeros((B, L, C // 32), dtype=torch.int32, device="cuda") for _ in range(NS)]
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=IND)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    if want("mask"):
        ms = _time(lambda i: cb.cawn_phase_accumulate_fwd(prm, ps[i % NS], g, t, ys[i % NS], ws, gate_mask=masks[i % NS]),
                   args.steps, args.warmup)
        _report("cfg1_train_fwd+mask", B * L, B * L * C * (16 + 0.125), ms, 1)
    if want("ear"):
        ew, eb = torch.randn((2 * cfg.H, 3), device="cuda"), torch.randn(2 * cfg.H, device="cuda")
        zs = [y.view(torch.float32).view(B, L, 2, C) for y in ys]      # planar rows are as long as interleaved ones
        ms = _time(lambda i: cb.cawn_phase_accumulate_fwd_ear(prm, ps[i % NS], g, t, ew, 3, zs[i % NS], ws, ear_bias=eb),
                   args.steps, args.warmup)
        _report("cfg1_train_fwd+ear_conv", B * L, B * L * C * 16, ms, 1)
    if want("bf16"):
        p16 = [p.view(torch.float32).to(torch.bfloat16).view(B, L, C, 2) for p in ps]
        y16 = [torch.empty((B, L, C, 2), dtype=torch.bfloat16, device="cuda") for _ in range(NS)]
        for name, fl, xin, yout, nbytes in (
                ("cfg1_train_fwd_bf16_in+out", cb.CAWN_FLAG_INPUT_BF16 | cb.CAWN_FLAG_OUTPUT_BF16, p16, y16, 8),
                ("cfg1_train_fwd_bf16_out", cb.CAWN_FLAG_OUTPUT_BF16, ps, y16, 12)):
            prm16 = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=IND | fl)
            ms = _time(lambda i: cb.cawn_phase_accumulate_fwd(prm16, xin[i % NS], g, t, yout[i % NS], ws), args.steps, args.warmup)
            _report(name, B * L, B * L * C * nbytes, ms, 1)
        del p16, y16
    if want("dynamic"):
        dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
        gl, fb = dev(dd["gamma_logit"]), dev(dd["freq_bias"])
        prm_d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=IND | cb.CAWN_FLAG_RETENTION_DYNAMIC)
        ws_d = cb.new_workspace(prm_d, cb.CAWN_OP_FWD)
        ms = _time(lambda i: cb.cawn_phase_accumulate_fwd(prm_d, ps[i % NS], None, t, ys[i % NS], ws_d, gamma_logit=gl, freq_bias=fb),
                   args.steps, args.warmup)
        assert cb.cawn_poll_status(ws_d) == 0
        _report("cfg1_train_fwd_dynamic_retention", B * L, B * L * (C * 16 + cfg.H * 4), ms, 1)
    assert cb.cawn_poll_status(ws) == 0
    del ps, ys, masks

    if want("cfg3"):
        _cfg3(args, cb, inputs, dev)
    if want("cfg4"):
        _cfg4(args, cb, inputs, dev, IND)
    if want("cfg4bwd"):
        _cfg4_bwd(args, cb, inputs, dev)
    if want("cfg2"):
        _cfg2(args, cb, inputs, dev, IND)
    if want("decode"):
        _decode(args, cb, inputs, dev)


def _decode(args, cb, inputs, dev):
    import torch
    # ---- single-token decode: L = 1 fused calls, state blob carried in place ------------------------
    cfg = inputs.CONFIGS[4]
    B, C, n = 1, cfg.C, 256
    d = inputs.fused_inputs(B, n, C, cfg.seed, cfg.conv_k)
    g, t, w = dev(d["gamma"]), dev(d["theta"]), dev(d["conv_w"])
    prm = cb.make_params(B, 1, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=float(inputs.gate_tau(cfg.gate_eps)),
                         conv_k=cfg.conv_k)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    nbytes = cb.cawn_workspace_bytes(prm, cb.CAWN_OP_STATE)
    blob = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    h = dev(d["h"])
    rows = [h[:, i:i + 1].contiguous() for i in range(n)]
    y = torch.empty((B, 1, C), dtype=torch.complex64, device="cuda")

    def gen(i):
        for j in range(n):
            cb.cawn_phase_accumulate_fwd(prm, rows[j], g, t, y, ws, conv_w=w, state_in=blob, state_out=blob)
    ms = _time(gen, max(args.steps // 10, 3), 2)
    assert cb.cawn_poll_status(ws) == 0
    _report("decode_fused_B1_L1", n, n * C * 12, ms, n, {"us_per_token": ms * 1e3 / n,
            "note": "one launch per token; latency-bound, bandwidth figures are not meaningful"})
    # the same n steps recorded once into a CUDA graph and replayed
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        gen(0)
    ms = _time(lambda i: graph.replay(), max(args.steps // 10, 3), 2)
    assert cb.cawn_poll_status(ws) == 0
    _report("decode_fused_B1_L1_cuda_graph", n, n * C * 12, ms, n, {"us_per_token": ms * 1e3 / n,
            "note": "256 decode steps replayed from one CUDA graph"})


def _cfg3(args, cb, inputs, dev):
    import torch
    # ---- config 3: backward with saved states ---------------------------------------------------
    cfg = inputs.CONFIGS[3]
    B, L, C = cfg.B, cfg.L, cfg.C
    d = inputs.config_inputs(cfg)
    g, t = dev(d["gamma"]), dev(d["theta"])
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps)
    NS = 3
    P = torch.empty((B, L, C), dtype=torch.complex64, device="cuda")
    wf = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    cb.cawn_phase_accumulate_fwd(prm, dev(d["p"]), g, t, P, wf)
    Ps = [P.clone() for _ in range(NS)]
    gys = [dev(d["grad_y"]) for _ in range(NS)]
    gps = [torch.empty_like(P) for _ in range(NS)]
    gg, gt = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    gsi = torch.empty((B, C), dtype=torch.complex64, device="cuda")
    wb = cb.new_workspace(prm, cb.CAWN_OP_BWD_SAVED)
    ms = _time(lambda i: cb.cawn_phase_accumulate_bwd(prm, Ps[i % NS], cb.CAWN_SAVED_STATES, g, t, gys[i % NS], gps[i % NS],
                                                      wb, grad_gamma=gg, grad_theta=gt, grad_state_in=gsi),
               args.steps, args.warmup)
    assert cb.cawn_poll_status(wb) == 0
    _report("cfg3_bwd", B * L, B * L * C * 24, ms, 2, {"note": "reads grad_y and saved P, writes grad_p; plus the finalize kernel"})
    # the same backward with time-varying retention (logit and frequency-bias gradients)
    dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
    gl, fb = dev(dd["gamma_logit"]), dev(dd["freq_bias"])
    prm_d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
    ggl, gfb = torch.empty((B, L, cfg.H), device="cuda"), torch.empty(cfg.F, device="cuda")
    ms = _time(lambda i: cb.cawn_phase_accumulate_bwd_dynamic(prm_d, Ps[i % NS], cb.CAWN_SAVED_STATES, gl, fb, t, gys[i % NS],
                                                              gps[i % NS], wb, grad_gamma_logit=ggl, grad_freq_bias=gfb,
                                                              grad_theta=gt, grad_state_in=gsi),
               args.steps, args.warmup)
    assert cb.cawn_poll_status(wb) == 0
    _report("cfg3_bwd_dynamic_retention", B * L, B * L * (C * 24 + cfg.H * 8), ms, 4,
            {"note": "memset of the logit gradient, scan (atomic adds per row and head), two reductions"})


def _cfg4(args, cb, inputs, dev, IND):
    import torch
    # ---- config 4: fused mixing path -------------------------------------------------------------
    cfg = inputs.CONFIGS[4]
    B, L, C = (args.cfg4_batch or cfg.B), cfg.L, cfg.C
    d = inputs.fused_inputs(B, L, C, cfg.seed, cfg.conv_k, cfg.gamma_lo, cfg.gamma_hi)
    g, t, w = dev(d["gamma"]), dev(d["theta"]), dev(d["conv_w"])
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=float(inputs.gate_tau(cfg.gate_eps)),
                         conv_k=cfg.conv_k, flags=IND)
    NS = 2
    hs = [dev(d["h"]) for _ in range(NS)]
    ys = [torch.empty((B, L, C), dtype=torch.complex64, device="cuda") for _ in range(NS)]
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    ms = _time(lambda i: cb.cawn_phase_accumulate_fwd(prm, hs[i % NS], g, t, ys[i % NS], ws, conv_w=w),
               max(args.steps // 2, 5), args.warmup)
    assert cb.cawn_poll_status(ws) == 0
    _report("cfg4_fused" if B == cfg.B else "cfg4_fused_B%d" % B, B * L, B * L * C * 12, ms, 1)
    if "dynamic" in args.only or not args.only:
        dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
        gl, fb = dev(dd["gamma_logit"]), dev(dd["freq_bias"])
        prm_d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=float(inputs.gate_tau(cfg.gate_eps)),
                               conv_k=cfg.conv_k, flags=IND | cb.CAWN_FLAG_RETENTION_DYNAMIC)
        ms = _time(lambda i: cb.cawn_phase_accumulate_fwd(prm_d, hs[i % NS], None, t, ys[i % NS], ws, conv_w=w,
                                                          gamma_logit=gl, freq_bias=fb),
                   max(args.steps // 2, 5), args.warmup)
        assert cb.cawn_poll_status(ws) == 0
        _report("cfg4_fused_dynamic_retention", B * L, B * L * (C * 12 + cfg.H * 4), ms, 1)
        # ... and with the Ear's convolution across the harmonics as the epilogue: the whole mixing step
        ew, eb = torch.randn((2 * cfg.H, 3), device="cuda"), torch.randn(2 * cfg.H, device="cuda")
        zs = [y.view(torch.float32).view(B, L, 2, C) for y in ys]
        ms = _time(lambda i: cb.cawn_phase_accumulate_fwd_ear(prm_d, hs[i % NS], None, t, ew, 3, zs[i % NS], ws, ear_bias=eb,
                                                              conv_w=w, gamma_logit=gl, freq_bias=fb),
                   max(args.steps // 2, 5), args.warmup)
        assert cb.cawn_poll_status(ws) == 0
        _report("cfg4_fused_dynamic_retention+ear_conv", B * L, B * L * (C * 12 + cfg.H * 4), ms, 1)
    if "bf16" in args.only or not args.only:
        prm16 = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=float(inputs.gate_tau(cfg.gate_eps)),
                               conv_k=cfg.conv_k, flags=IND | cb.CAWN_FLAG_INPUT_BF16 | cb.CAWN_FLAG_OUTPUT_BF16)
        h16 = [h.to(torch.bfloat16) for h in hs]
        y16 = [torch.empty((B, L, C, 2), dtype=torch.bfloat16, device="cuda") for _ in range(NS)]
        ms = _time(lambda i: cb.cawn_phase_accumulate_fwd(prm16, h16[i % NS], g, t, y16[i % NS], ws, conv_w=w),
                   max(args.steps // 2, 5), args.warmup)
        assert cb.cawn_poll_status(ws) == 0
        _report("cfg4_fused_bf16_in+out", B * L, B * L * C * 6, ms, 1)


def _cfg4_bwd(args, cb, inputs, dev):
    import torch
    # ---- config 4, backward of the fused mixing path (saved states) -------------------------------
    cfg = inputs.CONFIGS[4]
    B, L, C = (args.cfg4_batch or cfg.B), cfg.L, cfg.C
    d = inputs.fused_inputs(B, L, C, cfg.seed, cfg.conv_k, cfg.gamma_lo, cfg.gamma_hi)
    g, t, w, h = dev(d["gamma"]), dev(d["theta"]), dev(d["conv_w"]), dev(d["h"])
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=float(inputs.gate_tau(cfg.gate_eps)),
                         conv_k=cfg.conv_k)
    P = torch.empty((B, L, C), dtype=torch.complex64, device="cuda")
    wf = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    cb.cawn_phase_accumulate_fwd(prm, h, g, t, P, wf, conv_w=w)
    gy = torch.randn((B, L, C, 2), device="cuda").view(torch.float32)
    gy = torch.view_as_complex(gy)
    gh = torch.empty((B, L, C), device="cuda")
    gw, gb = torch.empty((C, cfg.conv_k), device="cuda"), torch.empty(C, device="cuda")
    gg, gt = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    wb = cb.new_workspace(prm, cb.CAWN_OP_MIXING_BWD)
    ms = _time(lambda i: cb.cawn_mixing_bwd(prm, h, w, g, t, gy, gh, wb, saved_states=P, grad_conv_w=gw,
                                            grad_conv_bias=gb, grad_gamma=gg, grad_theta=gt),
               max(args.steps // 2, 5), args.warmup)
    assert cb.cawn_poll_status(wb) == 0
    # reads grad_y (8) + P (8) + h (4), writes grad_h (4)
    _report("cfg4_mixing_bwd" if B == cfg.B else "cfg4_mixing_bwd_B%d" % B, B * L, B * L * C * 24, ms, 4,
            {"note": "reverse scan with the prelude backward as its epilogue, seam rows, two reductions"})
    # the same with time-varying retention (the paper's layer form)
    dd = inputs.dynamic_retention_inputs(B, L, cfg.H, cfg.F, 7)
    gl, fb = dev(dd["gamma_logit"]), dev(dd["freq_bias"])
    prm_d = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=float(inputs.gate_tau(cfg.gate_eps)),
                           conv_k=cfg.conv_k, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
    cb.cawn_phase_accumulate_fwd(prm_d, h, None, t, P, wf, conv_w=w, gamma_logit=gl, freq_bias=fb)
    ggl, gfb = torch.empty((B, L, cfg.H), device="cuda"), torch.empty(cfg.F, device="cuda")
    ms = _time(lambda i: cb.cawn_mixing_bwd_dynamic(prm_d, h, w, gl, fb, t, gy, gh, wb, saved_states=P, grad_conv_w=gw,
                                                    grad_conv_bias=gb, grad_gamma_logit=ggl, grad_freq_bias=gfb, grad_theta=gt),
               max(args.steps // 2, 5), args.warmup)
    assert cb.cawn_poll_status(wb) == 0
    _report("cfg4_mixing_bwd_dynamic_retention" if B == cfg.B else "cfg4_mixing_bwd_dynamic_retention_B%d" % B, B * L,
            B * L * (C * 24 + cfg.H * 8), ms, 6, {"note": "plus the memset of the logit gradient and the frequency-bias reduction"})


def _cfg2(args, cb, inputs, dev, IND):
    import torch
    # ---- config 2: chunked prefill, 64 calls of 4096 tokens with the state carried ---------------
    cfg = inputs.CONFIGS[2]
    C, n = cfg.C, cfg.chunk
    stream = inputs.prefill_stream(cfg, total=16 * n)
    gamma, theta = next(stream)
    g, t = dev(gamma), dev(theta)
    chunks = [dev(p) for p in stream]                     # 16 distinct chunks (805 MB), cycled
    ys = [torch.empty_like(chunks[0]) for _ in range(4)]
    state = torch.zeros((cfg.B, C), dtype=torch.complex64, device="cuda")
    prm = cb.make_params(cfg.B, n, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=IND)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    ncalls = 64

    def prefill(i):
        for j in range(ncalls):
            cb.cawn_phase_accumulate_fwd(prm, chunks[j % 16], g, t, ys[j % 4], ws, state_in=state, state_out=state)
    ms = _time(prefill, max(args.steps // 10, 3), 2)
    assert cb.cawn_poll_status(ws) == 0
    _report("cfg2_chunked_prefill", ncalls * n, ncalls * n * C * 16, ms, ncalls,
            {"us_per_4096_token_call": ms * 1e3 / ncalls, "note": "one launch per chunk, state carried on the device"})
    # the same 64 calls recorded once into a CUDA graph: takes the host's per-call cost out
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        prefill(0)
    ms = _time(lambda i: graph.replay(), max(args.steps // 10, 3), 2)
    assert cb.cawn_poll_status(ws) == 0
    _report("cfg2_chunked_prefill_cuda_graph", ncalls * n, ncalls * n * C * 16, ms, ncalls,
            {"us_per_4096_token_call": ms * 1e3 / ncalls, "note": "64 chunk calls replayed from one CUDA graph"})


if __name__ == "__main__":
    sys.exit(main())
