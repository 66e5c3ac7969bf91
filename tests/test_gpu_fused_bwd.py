"""GPU parity: backward of the fused Resonance mixing path (cawn_mixing_bwd) against the oracle's
fused_backward: gradients of the hidden states, conv weights and bias, retention, rotation, and
of the carried state and conv history."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err

TOL = 1e-4


def run_mixing_bwd(d, eps, clamp_silu=False, P_in=None, gso_P=None, gso_tail=None, want_param=True):
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    h, w = d["h"], d["conv_w"]
    B, L, C = h.shape
    Kc = w.shape[1]
    tau = float(inputs.gate_tau(eps))
    flags = cb.CAWN_FLAG_PRELUDE_CLAMP_SILU if clamp_silu else 0
    prm = cb.make_params(B, L, 1, C, gate_eps=eps, gate_tau=tau, conv_k=Kc, flags=flags)
    g, t, dw_, db_ = dev(d["gamma"]), dev(d["theta"]), dev(w), dev(d.get("conv_bias"))
    s_in, off = state_blob(B, C, Kc, P_in, d.get("tail_in"))
    have_state = P_in is not None or d.get("tail_in") is not None
    # forward (unclamped) to get the states a training step would have saved
    y = torch.empty((B, L, C), dtype=torch.complex64, device="cuda")
    wf = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    cb.cawn_phase_accumulate_fwd(prm, dev(h), g, t, y, wf, conv_w=dw_, conv_bias=db_,
                                 state_in=s_in if have_state else None)
    assert cb.cawn_poll_status(wf) == 0
    gso, _ = state_blob(B, C, Kc, gso_P, gso_tail)
    have_gso = gso_P is not None or gso_tail is not None
    ws = cb.new_workspace(prm, cb.CAWN_OP_MIXING_BWD)
    nan = float("nan")
    gh = torch.full((B, L, C), nan, device="cuda")
    gw = torch.full((C, Kc), nan, device="cuda") if want_param else None
    gb = torch.full((C,), nan, device="cuda") if want_param else None
    gg = torch.full((C,), nan, device="cuda") if want_param else None
    gt = torch.full((C,), nan, device="cuda") if want_param else None
    gsi, _ = state_blob(B, C, Kc)
    gsi.fill_(0xFF)
    cb.cawn_mixing_bwd(prm, dev(h), dw_, g, t, dev(d["G"]), gh, ws, conv_bias=db_, saved_states=y if want_param else None,
                       state_in=s_in if have_state else None, grad_state_out=gso if have_gso else None,
                       grad_conv_w=gw, grad_conv_bias=gb, grad_gamma=gg, grad_theta=gt, grad_state_in=gsi)
    assert cb.cawn_poll_status(ws) == 0
    dP, dtail = split_blob(gsi, off, B, C, Kc)
    out = {"dh": gh.cpu().numpy(), "dstate_in": dP.copy(), "dtail_in": dtail.copy()}
    if want_param:
        out.update(dw=gw.cpu().numpy(), dbias=gb.cpu().numpy(), dgamma=gg.cpu().numpy(), dtheta=gt.cpu().numpy())
    return out


def reference(d, eps, clamp_silu=False, P_in=None, gso_P=None, gso_tail=None):
    si = None if P_in is None else P_in.astype(np.complex128)
    dso = None if gso_P is None else gso_P.astype(np.complex128)
    return oracle.fused_backward(d["h"], d["conv_w"], d["gamma"], d["theta"], d["G"], eps, inputs.gate_tau(eps),
                                 bias=d.get("conv_bias"), clamp_silu=clamp_silu, tail_in=d.get("tail_in"),
                                 state_in=si, dstate_out=dso, dtail_out=gso_tail)


def make(B, L, C, Kc, seed, with_tail=True, with_bias=True):
    d = inputs.fused_inputs(B, L, C, seed, conv_k=Kc, with_tail=with_tail and Kc > 1, with_bias=with_bias)
    rng = np.random.default_rng(seed + 7)
    d["G"] = (rng.normal(size=(B, L, C)) + 1j * rng.normal(size=(B, L, C))).astype(np.complex64)
    d["P_in"] = (rng.normal(0, 2, (B, C)) + 1j * rng.normal(0, 2, (B, C))).astype(np.complex64)
    d["gso_P"] = (rng.normal(size=(B, C)) + 1j * rng.normal(size=(B, C))).astype(np.complex64)
    d["gso_tail"] = rng.normal(size=(B, max(Kc - 1, 0), C)).astype(np.float32)
    return d


def compare(got, ref, L, Kc):
    if L:
        assert not np.isnan(got["dh"]).any()
        assert floored_rel_err(got["dh"], ref["dh"], axes=(0, 1)) < TOL
    assert floored_rel_err(got["dstate_in"], ref["dstate_in"]) < TOL
    if Kc > 1:
        assert floored_rel_err(got["dtail_in"], ref["dtail_in"], axes=None) < TOL
    for k in ("dw", "dbias", "dgamma", "dtheta"):
        if k in got:
            assert not np.isnan(got[k]).any(), k
            assert floored_rel_err(got[k], ref[k]) < TOL, k


@pytest.mark.parametrize("B,L,C,Kc", [(1, 1, 64, 4), (2, 2, 64, 4), (1, 3, 64, 3), (2, 17, 64, 4), (1, 128, 64, 4),
                                      (2, 129, 128, 3), (2, 300, 192, 4), (1, 1000, 64, 2), (2, 257, 100, 4),
                                      (1, 140, 33, 4), (1, 200, 64, 1), (1, 515, 768, 4)])
def test_mixing_bwd_shapes(B, L, C, Kc):
    d = make(B, L, C, Kc, seed=800 + L + C)
    tail = d["gso_tail"] if Kc > 1 else None
    got = run_mixing_bwd(d, 0.1, P_in=d["P_in"], gso_P=d["gso_P"], gso_tail=tail)
    compare(got, reference(d, 0.1, P_in=d["P_in"], gso_P=d["gso_P"], gso_tail=tail), L, Kc)


def test_mixing_bwd_taps_only_8_byte_aligned(monkeypatch):
    from test_gpu_fused import taps_at_8_byte_offset
    taps_at_8_byte_offset(monkeypatch)
    d = make(2, 300, 192, 4, seed=1492)
    got = run_mixing_bwd(d, 0.1, P_in=d["P_in"], gso_P=d["gso_P"], gso_tail=d["gso_tail"])
    compare(got, reference(d, 0.1, P_in=d["P_in"], gso_P=d["gso_P"], gso_tail=d["gso_tail"]), 300, 4)


@pytest.mark.parametrize("L", [15, 16, 17, 18, 19, 31, 32, 33, 34, 35, 63, 64, 65, 66, 67, 127, 128, 129, 130, 131, 192, 193])
def test_mixing_bwd_rows_at_tile_seams(L):
    """Lengths around multiples of the tile (16 rows up to L = 32, 64 beyond): the rows whose conv
    transpose crosses a tile seam, a last tile of one to three rows, and the history gradient."""
    d = make(2, L, 66, 4, seed=1200 + L)
    got = run_mixing_bwd(d, 0.1, P_in=d["P_in"], gso_P=d["gso_P"], gso_tail=d["gso_tail"])
    compare(got, reference(d, 0.1, P_in=d["P_in"], gso_P=d["gso_P"], gso_tail=d["gso_tail"]), L, 4)


def test_mixing_bwd_clamp_silu_and_no_state():
    d = make(2, 400, 128, 4, seed=91, with_tail=False)
    d["h"] = (d["h"] * 20).astype(np.float32)
    got = run_mixing_bwd(d, 0.1, clamp_silu=True)
    compare(got, reference(d, 0.1, clamp_silu=True), 400, 4)


def test_mixing_bwd_without_parameter_gradients():
    d = make(2, 300, 64, 4, seed=92)
    got = run_mixing_bwd(d, 0.1, P_in=d["P_in"], want_param=False)
    compare(got, reference(d, 0.1, P_in=d["P_in"]), 300, 4)


def test_mixing_bwd_repeatable_bitwise():
    d = make(2, 700, 128, 4, seed=93)
    a = run_mixing_bwd(d, 0.1, P_in=d["P_in"])
    b = run_mixing_bwd(d, 0.1, P_in=d["P_in"])
    for k in a:
        assert np.array_equal(a[k].view(np.uint32), b[k].view(np.uint32)), k


def test_mixing_bwd_config4_full_size():
    """Config 4 at full size (B=16, L=8192, C=768), the launch configuration the bench times: the
    hidden-state gradient and the state gradient of all sixteen batch rows, and the gradients of
    the conv weights, retention and rotation.  The oracle walks the rows one by one; a parameter
    gradient is a sum over the batch, so the rows' fp64 results are added up."""
    cfg = inputs.CONFIGS[4]
    B = cfg.B
    d = make(B, cfg.L, cfg.C, cfg.conv_k, seed=cfg.seed, with_tail=False, with_bias=False)
    got = run_mixing_bwd(d, cfg.gate_eps)
    sums = {k: 0.0 for k in ("dw", "dgamma", "dtheta")}
    for b in range(B):
        sub = {k: (v[b:b + 1] if k in ("h", "G") else v) for k, v in d.items()}
        ref = reference(sub, cfg.gate_eps)
        assert floored_rel_err(got["dh"][b:b + 1], ref["dh"], axes=(0, 1)) < TOL, b
        assert floored_rel_err(got["dstate_in"][b:b + 1], ref["dstate_in"]) < TOL, b
        assert floored_rel_err(got["dtail_in"][b:b + 1], ref["dtail_in"], axes=None) < TOL, b
        for k in sums:
            sums[k] = sums[k] + ref[k].astype(np.float64)
    for k in sums:
        assert floored_rel_err(got[k], sums[k]) < TOL, k


@pytest.mark.parametrize("B,L,H,F,Kc", [(1, 1, 1, 64, 4), (2, 70, 2, 64, 4), (1, 200, 3, 32, 3), (2, 131, 5, 16, 4), (1, 300, 3, 11, 4),
                                        (1, 515, 12, 64, 4), (2, 20, 2, 64, 2)])
def test_mixing_bwd_with_dynamic_retention(B, L, H, F, Kc):
    """Backward of the paper's own layer form: conv prelude, gated push, retention per token and head."""
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    C = H * F
    d = make(B, L, C, Kc, seed=1500 + L)
    d.update(inputs.dynamic_retention_inputs(B, L, H, F, 1501 + L))
    eps, tau = 0.1, float(inputs.gate_tau(0.1))
    tail = d["gso_tail"] if Kc > 1 else None
    ref = oracle.fused_backward(d["h"], d["conv_w"], None, d["theta"], d["G"], eps, tau, bias=d.get("conv_bias"),
                                tail_in=d.get("tail_in"), state_in=d["P_in"].astype(np.complex128),
                                dstate_out=d["gso_P"].astype(np.complex128), dtail_out=tail,
                                gamma_logit=d["gamma_logit"], freq_bias=d["freq_bias"], H=H)
    prm = cb.make_params(B, L, H, F, gate_eps=eps, gate_tau=tau, conv_k=Kc, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
    t, w, bias = dev(d["theta"]), dev(d["conv_w"]), dev(d.get("conv_bias"))
    gl, fb = dev(d["gamma_logit"]), dev(d["freq_bias"])
    s_in, off = state_blob(B, C, Kc, d["P_in"], d.get("tail_in"))
    y = torch.empty((B, L, C), dtype=torch.complex64, device="cuda")
    wf = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    cb.cawn_phase_accumulate_fwd(prm, dev(d["h"]), None, t, y, wf, conv_w=w, conv_bias=bias, gamma_logit=gl, freq_bias=fb,
                                 state_in=s_in)
    assert cb.cawn_poll_status(wf) == 0
    gso, _ = state_blob(B, C, Kc, d["gso_P"], tail)
    gsi, _ = state_blob(B, C, Kc)
    ws = cb.new_workspace(prm, cb.CAWN_OP_MIXING_BWD)
    nan = float("nan")
    gh = torch.full((B, L, C), nan, device="cuda")
    gw, gb = torch.full((C, Kc), nan, device="cuda"), torch.full((C,), nan, device="cuda")
    ggl, gfb, gt = torch.full((B, L, H), nan, device="cuda"), torch.full((F,), nan, device="cuda"), torch.full((C,), nan, device="cuda")
    cb.cawn_mixing_bwd_dynamic(prm, dev(d["h"]), w, gl, fb, t, dev(d["G"]), gh, ws, conv_bias=bias, saved_states=y, state_in=s_in,
                               grad_state_out=gso, grad_conv_w=gw, grad_conv_bias=gb, grad_gamma_logit=ggl, grad_freq_bias=gfb,
                               grad_theta=gt, grad_state_in=gsi)
    assert cb.cawn_poll_status(ws) == 0
    dP, dtail = split_blob(gsi, off, B, C, Kc)
    assert floored_rel_err(gh.cpu().numpy(), ref["dh"], axes=(0, 1)) < TOL
    assert floored_rel_err(gw.cpu().numpy(), ref["dw"]) < TOL
    assert floored_rel_err(gb.cpu().numpy(), ref["dbias"]) < TOL
    assert floored_rel_err(ggl.cpu().numpy(), ref["dgamma_logit"]) < TOL
    assert floored_rel_err(gfb.cpu().numpy(), ref["dfreq_bias"]) < TOL
    assert floored_rel_err(gt.cpu().numpy(), ref["dtheta"]) < TOL
    assert floored_rel_err(dP, ref["dstate_in"]) < TOL
    if Kc > 1:
        assert floored_rel_err(dtail, ref["dtail_in"], axes=None) < TOL
