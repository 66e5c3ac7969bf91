"""GPU parity: the forward with the Ear's depthwise convolution across the harmonics as its
epilogue (cawn_phase_accumulate_fwd_ear) against oracle.forward / fused_forward + oracle.ear_conv."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err

TOL = 1e-4


def ear_taps(H, Ke, seed, bias=True):
    rng = np.random.default_rng(seed)
    w = rng.normal(0, 0.6, (2 * H, Ke)).astype(np.float32)
    b = rng.normal(0, 0.3, 2 * H).astype(np.float32) if bias else None
    return w, b


def run_ear(B, L, H, F, Ke, seed, fused=False, clamp_abs=0.0, bias=True, with_state=True, want_mask=True):
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    C = H * F
    ew, eb = ear_taps(H, Ke, seed + 1, bias)
    eps = 0.1
    rng = np.random.default_rng(seed + 2)
    P_in = (rng.normal(0, 2, (B, C)) + 1j * rng.normal(0, 2, (B, C))).astype(np.complex64) if with_state else None
    MW = (C + 31) // 32
    d_m = torch.zeros((B, L, MW), dtype=torch.int32, device="cuda") if want_mask else None
    z = torch.full((B, L, 2, H, F), float("nan"), device="cuda")
    if fused:
        Kc = 4
        d = inputs.fused_inputs(B, L, C, seed, conv_k=Kc, with_tail=with_state)
        tau = float(inputs.gate_tau(eps))
        prm = cb.make_params(B, L, H, F, gate_eps=eps, gate_tau=tau, clamp_abs=clamp_abs, conv_k=Kc)
        s_in, off = state_blob(B, C, Kc, P_in, d.get("tail_in"))
        s_out, _ = state_blob(B, C, Kc)
        ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
        cb.cawn_phase_accumulate_fwd_ear(prm, dev(d["h"]), dev(d["gamma"]), dev(d["theta"]), dev(ew), Ke, z, ws,
                                         ear_bias=dev(eb), conv_w=dev(d["conv_w"]), conv_bias=dev(d.get("conv_bias")),
                                         state_in=s_in if with_state else None, state_out=s_out, gate_mask=d_m)
        assert cb.cawn_poll_status(ws) == 0
        y, so, mask, _ = oracle.fused_forward(d["h"], d["conv_w"], d["gamma"], d["theta"], eps, tau, bias=d.get("conv_bias"),
                                              tail_in=d.get("tail_in"), state_in=None if P_in is None else P_in.astype(np.complex128),
                                              clamp_abs=clamp_abs)
        P_out, _ = split_blob(s_out, off, B, C, Kc)
    else:
        d = inputs.scan_inputs(B, L, C, seed)
        prm = cb.make_params(B, L, H, F, gate_eps=eps, clamp_abs=clamp_abs)
        ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
        d_so = torch.full((B, C), float("nan"), dtype=torch.complex64, device="cuda")
        cb.cawn_phase_accumulate_fwd_ear(prm, dev(d["p"]), dev(d["gamma"]), dev(d["theta"]), dev(ew), Ke, z, ws,
                                         ear_bias=dev(eb), state_in=dev(P_in), state_out=d_so, gate_mask=d_m)
        assert cb.cawn_poll_status(ws) == 0
        y, so, mask = oracle.forward(d["p"], d["gamma"], d["theta"], eps, clamp_abs=clamp_abs,
                                     state_in=None if P_in is None else P_in.astype(np.complex128))
        P_out = d_so.cpu().numpy()
    ref = oracle.ear_conv(y, ew, eb, H, F)
    got = z.cpu().numpy()
    if L:
        assert not np.isnan(got).any()
        assert floored_rel_err(got, ref) < TOL
        assert floored_rel_err(P_out, so) < TOL          # the carried state stays unconvolved
    return got, ref


@pytest.mark.parametrize("B,L,H,F,Ke", [(1, 1, 1, 64, 3), (2, 37, 2, 32, 3), (1, 130, 4, 16, 3), (2, 300, 3, 64, 3),
                                        (1, 257, 12, 64, 3), (2, 100, 5, 8, 3), (1, 200, 7, 9, 3), (1, 150, 3, 11, 3),
                                        (2, 140, 64, 1, 3), (1, 129, 2, 64, 1), (1, 1000, 1, 50, 3), (2, 64, 3, 2, 3)])
def test_ear_cartesian_shapes(B, L, H, F, Ke):
    if H * F > 64 and 64 % F != 0:
        pytest.skip("harmonics would straddle channel groups")
    run_ear(B, L, H, F, Ke, seed=300 + L + H)


@pytest.mark.parametrize("B,L,H,F", [(1, 5, 1, 64), (2, 200, 2, 64), (1, 333, 3, 32), (1, 131, 1, 33)])
def test_ear_fused_shapes(B, L, H, F):
    run_ear(B, L, H, F, 3, seed=400 + L, fused=True)


def test_ear_sees_the_clamped_state():
    run_ear(2, 400, 2, 64, 3, seed=55, clamp_abs=1.5)


def test_ear_without_bias_state_or_mask():
    run_ear(1, 260, 2, 64, 3, seed=56, bias=False, with_state=False, want_mask=False)


def test_identity_tap_gives_planar_z_bitwise():
    """ear_k = 1, tap 1, no bias: z_conv is the interleaved output's real parts, then its imaginary parts."""
    import torch
    from gpu_util import dev, run_fwd
    from paper_2604_04250_b200 import binding as cb
    B, L, H, F = 2, 300, 2, 64
    d = inputs.scan_inputs(B, L, H * F, 77)
    y, _, _ = run_fwd(d["p"], d["gamma"], d["theta"], 0.1, H=H)
    prm = cb.make_params(B, L, H, F, gate_eps=0.1)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    z = torch.empty((B, L, 2, H * F), device="cuda")
    cb.cawn_phase_accumulate_fwd_ear(prm, dev(d["p"]), dev(d["gamma"]), dev(d["theta"]),
                                     torch.ones((2 * H, 1), device="cuda"), 1, z, ws)
    assert cb.cawn_poll_status(ws) == 0
    z = z.cpu().numpy()
    # tap * value + 0 is exact
    assert np.array_equal(z[:, :, 0].view(np.uint32), np.ascontiguousarray(y.real).view(np.uint32))
    assert np.array_equal(z[:, :, 1].view(np.uint32), np.ascontiguousarray(y.imag).view(np.uint32))


def test_ear_refusals():
    import torch
    from paper_2604_04250_b200 import binding as cb
    one = torch.ones(64, device="cuda")
    z = torch.empty((1, 4, 2, 3, 48), device="cuda")
    prm = cb.make_params(1, 4, 3, 48)                      # 48 does not divide 64 and C > 64
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    x = torch.zeros((1, 4, 144), dtype=torch.complex64, device="cuda")
    g = torch.ones(144, device="cuda")
    with pytest.raises(cb.CawnError) as e:
        cb.cawn_phase_accumulate_fwd_ear(prm, x, g, g, one, 3, z, ws)
    assert e.value.status == cb.CAWN_ERR_UNSUPPORTED
    prm = cb.make_params(1, 4, 3, 32)
    with pytest.raises(cb.CawnError) as e:
        cb.cawn_phase_accumulate_fwd_ear(prm, x, g, g, one, 5, z, ws)
    assert e.value.status == cb.CAWN_ERR_UNSUPPORTED


@pytest.mark.parametrize("B,L,H,F,fused", [(2, 200, 2, 64, True), (1, 333, 3, 32, True), (1, 515, 12, 64, True),
                                            (2, 150, 4, 16, False), (1, 20, 1, 64, True)])
def test_ear_with_dynamic_retention(B, L, H, F, fused):
    """The whole Resonance mixing step in one kernel: (conv prelude, gated push,) recurrence with
    per-token retention, clamp, Ear convolution across the harmonics."""
    import torch
    from gpu_util import dev, state_blob
    from paper_2604_04250_b200 import binding as cb
    C = H * F
    eps, clamp = 0.1, 3.0
    ew, eb = ear_taps(H, 3, 810 + L)
    dd = inputs.dynamic_retention_inputs(B, L, H, F, 811 + L)
    gl, fb = dev(dd["gamma_logit"]), dev(dd["freq_bias"])
    z = torch.full((B, L, 2, H, F), float("nan"), device="cuda")
    kw = dict(gamma_logit=dd["gamma_logit"], freq_bias=dd["freq_bias"], H=H)
    if fused:
        Kc = 4
        d = inputs.fused_inputs(B, L, C, 812 + L, conv_k=Kc, with_tail=True)
        tau = float(inputs.gate_tau(eps))
        prm = cb.make_params(B, L, H, F, gate_eps=eps, gate_tau=tau, clamp_abs=clamp, conv_k=Kc, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
        s_in, _ = state_blob(B, C, Kc, None, d["tail_in"])
        ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
        cb.cawn_phase_accumulate_fwd_ear(prm, dev(d["h"]), None, dev(d["theta"]), dev(ew), 3, z, ws, ear_bias=dev(eb),
                                         conv_w=dev(d["conv_w"]), conv_bias=dev(d.get("conv_bias")), gamma_logit=gl,
                                         freq_bias=fb, state_in=s_in)
        y, _, _, _ = oracle.fused_forward(d["h"], d["conv_w"], None, d["theta"], eps, tau, bias=d.get("conv_bias"),
                                          tail_in=d["tail_in"], clamp_abs=clamp, **kw)
    else:
        d = inputs.scan_inputs(B, L, C, 813 + L)
        prm = cb.make_params(B, L, H, F, gate_eps=eps, clamp_abs=clamp, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
        ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
        cb.cawn_phase_accumulate_fwd_ear(prm, dev(d["p"]), None, dev(d["theta"]), dev(ew), 3, z, ws, ear_bias=dev(eb),
                                         gamma_logit=gl, freq_bias=fb)
        zz, _ = oracle.gate(d["p"], eps)
        y, _ = oracle.scan(zz, d["theta"], clamp_abs=clamp, **kw)
    assert cb.cawn_poll_status(ws) == 0
    assert floored_rel_err(z.cpu().numpy(), oracle.ear_conv(y, ew, eb, H, F)) < TOL
