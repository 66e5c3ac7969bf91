"""GPU parity: the paper's time-varying retention gamma_t = sigmoid(logit[b,t,h] + bias[k]),
forward and backward, through the C ABI against the fp64 oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err, unpack_mask

TOL = 1e-4


def make(B, L, H, F, seed, with_grad=False):
    d = inputs.scan_inputs(B, L, H * F, seed=seed, with_state=True, with_grad=with_grad)
    d.update(inputs.dynamic_retention_inputs(B, L, H, F, seed + 1))
    return d


def run_fwd_dyn(d, H, F, eps, use_state=True, clamp_abs=0.0):
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    B, L, C = d["p"].shape
    prm = cb.make_params(B, L, H, F, gate_eps=eps, clamp_abs=clamp_abs, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    y = torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda")
    so = torch.full((B, C), float("nan"), dtype=torch.complex64, device="cuda")
    m = torch.zeros((B, L, (C + 31) // 32), dtype=torch.int32, device="cuda")
    cb.cawn_phase_accumulate_fwd(prm, dev(d["p"]), None, dev(d["theta"]), y, ws, gamma_logit=dev(d["gamma_logit"]),
                                 freq_bias=dev(d["freq_bias"]), state_in=dev(d["state_in"]) if use_state else None,
                                 state_out=so, gate_mask=m)
    assert cb.cawn_poll_status(ws) == 0
    return y, so.cpu().numpy(), m.cpu().numpy().view(np.uint32)


def ref_fwd(d, eps, use_state=True, clamp_abs=0.0, want_P=False):
    z, mask = oracle.gate(d["p"], eps)
    si = d["state_in"].astype(np.complex128) if use_state else None
    out = oracle.scan(z, d["theta"], gamma_logit=d["gamma_logit"], freq_bias=d["freq_bias"], state_in=si,
                      clamp_abs=clamp_abs, want_P=want_P)
    return z, mask, out


@pytest.mark.parametrize("B,L,H,F", [(1, 1, 1, 64), (2, 5, 4, 16), (1, 256, 4, 16), (2, 129, 2, 64), (1, 1000, 3, 64),
                                     (2, 300, 1, 192), (1, 515, 12, 64), (2, 200, 5, 20), (1, 140, 3, 11)])
def test_dynamic_forward_shapes(B, L, H, F):
    d = make(B, L, H, F, seed=500 + L + F)
    _, m_ref, (y_ref, so_ref) = ref_fwd(d, 0.1)
    y, so, mw = run_fwd_dyn(d, H, F, 0.1)
    assert np.array_equal(unpack_mask(mw, H * F), m_ref)
    assert floored_rel_err(y.cpu().numpy(), y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so, so_ref) < TOL


def test_dynamic_forward_training_shape():
    cfg = inputs.CONFIGS[1]
    d = make(cfg.B, cfg.L, cfg.H, cfg.F, seed=77)
    _, m_ref, (y_ref, so_ref) = ref_fwd(d, cfg.gate_eps, use_state=False)
    y, so, mw = run_fwd_dyn(d, cfg.H, cfg.F, cfg.gate_eps, use_state=False)
    assert np.array_equal(unpack_mask(mw, cfg.C), m_ref)
    assert floored_rel_err(y.cpu().numpy(), y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so, so_ref) < TOL


def run_bwd_dyn(d, H, F, eps, saved_kind):
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    B, L, C = d["p"].shape
    prm = cb.make_params(B, L, H, F, gate_eps=eps, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
    if saved_kind == cb.CAWN_SAVED_STATES:
        saved, _, _ = run_fwd_dyn(d, H, F, eps)
        op = cb.CAWN_OP_BWD_SAVED
    else:
        saved, op = dev(d["p"]), cb.CAWN_OP_BWD_PUSHES
    ws = cb.new_workspace(prm, op)
    nan = float("nan")
    gp = torch.full((B, L, C), nan, dtype=torch.complex64, device="cuda")
    ggl = torch.full((B, L, H), nan, device="cuda")
    gfb = torch.full((F,), nan, device="cuda")
    gth = torch.full((C,), nan, device="cuda")
    gsi = torch.full((B, C), nan, dtype=torch.complex64, device="cuda")
    cb.cawn_phase_accumulate_bwd_dynamic(prm, saved, saved_kind, dev(d["gamma_logit"]), dev(d["freq_bias"]),
                                         dev(d["theta"]), dev(d["grad_y"]), gp, ws, state_in=dev(d["state_in"]),
                                         grad_state_out=dev(d["grad_state_out"]), grad_gamma_logit=ggl,
                                         grad_freq_bias=gfb, grad_theta=gth, grad_state_in=gsi)
    assert cb.cawn_poll_status(ws) == 0
    return {k: v.cpu().numpy() for k, v in dict(dp=gp, dgamma_logit=ggl, dfreq_bias=gfb, dtheta=gth, dstate_in=gsi).items()}


@pytest.mark.parametrize("saved_kind", [0, 1])
@pytest.mark.parametrize("B,L,H,F", [(1, 1, 1, 64), (2, 5, 4, 16), (2, 65, 2, 64), (1, 300, 4, 16), (1, 700, 3, 64),
                                     (2, 333, 5, 20), (1, 2049, 12, 64), (2, 130, 1, 192)])
def test_dynamic_backward_shapes(B, L, H, F, saved_kind):
    d = make(B, L, H, F, seed=600 + L + F, with_grad=True)
    z, _ = oracle.gate(d["p"], 0.1)
    ref = oracle.scan_bwd(z, d["theta"], d["grad_y"], gamma_logit=d["gamma_logit"], freq_bias=d["freq_bias"],
                          state_in=d["state_in"].astype(np.complex128),
                          dstate_out=d["grad_state_out"].astype(np.complex128))
    got = run_bwd_dyn(d, H, F, 0.1, saved_kind)
    assert floored_rel_err(got["dp"], ref["dp"], axes=(0, 1)) < TOL
    assert floored_rel_err(got["dstate_in"], ref["dstate_in"]) < TOL
    for k in ("dgamma_logit", "dfreq_bias", "dtheta"):
        assert not np.isnan(got[k]).any(), k
        assert floored_rel_err(got[k], ref[k]) < TOL, k


@pytest.mark.parametrize("B,L,H,F,Kc", [(1, 3, 1, 64, 4), (2, 200, 2, 64, 4), (1, 333, 3, 32, 3), (2, 150, 5, 16, 4),
                                        (1, 131, 3, 11, 4), (1, 515, 12, 64, 4), (2, 20, 2, 64, 2)])
def test_fused_path_with_dynamic_retention(B, L, H, F, Kc):
    """The paper's own combination: conv prelude and gated push feeding a recurrence whose retention
    varies per token and head; chunked in two calls with the state blob carried."""
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    C = H * F
    d = inputs.fused_inputs(B, L, C, 700 + L, conv_k=Kc, with_tail=True)
    d.update(inputs.dynamic_retention_inputs(B, L, H, F, 701 + L))
    eps, tau = 0.1, float(inputs.gate_tau(0.1))
    rng = np.random.default_rng(9)
    P_in = (rng.normal(0, 2, (B, C)) + 1j * rng.normal(0, 2, (B, C))).astype(np.complex64)
    y_ref, so_ref, m_ref, tail_ref = oracle.fused_forward(
        d["h"], d["conv_w"], None, d["theta"], eps, tau, bias=d.get("conv_bias"), tail_in=d["tail_in"],
        state_in=P_in.astype(np.complex128), gamma_logit=d["gamma_logit"], freq_bias=d["freq_bias"], H=H)
    blob, off = state_blob(B, C, Kc, P_in, d["tail_in"])
    t, w, bias = dev(d["theta"]), dev(d["conv_w"]), dev(d.get("conv_bias"))
    fb = dev(d["freq_bias"])
    y = torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda")
    m = torch.zeros((B, L, (C + 31) // 32), dtype=torch.int32, device="cuda")
    cut = L // 2
    for lo, hi in ((0, cut), (cut, L)):
        n = hi - lo
        prm = cb.make_params(B, n, H, F, gate_eps=eps, gate_tau=tau, conv_k=Kc, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)
        ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
        yy = torch.full((B, n, C), float("nan"), dtype=torch.complex64, device="cuda")
        mm = torch.zeros((B, n, (C + 31) // 32), dtype=torch.int32, device="cuda")
        cb.cawn_phase_accumulate_fwd(prm, dev(d["h"][:, lo:hi]), None, t, yy, ws, conv_w=w, conv_bias=bias,
                                     gamma_logit=dev(d["gamma_logit"][:, lo:hi]), freq_bias=fb,
                                     state_in=blob, state_out=blob, gate_mask=mm)
        assert cb.cawn_poll_status(ws) == 0
        y[:, lo:hi] = yy
        m[:, lo:hi] = mm
    assert floored_rel_err(y.cpu().numpy(), y_ref) < TOL
    P_out, tail_out = split_blob(blob, off, B, C, Kc)
    assert floored_rel_err(P_out, so_ref) < TOL
    assert np.array_equal(tail_out, tail_ref.astype(np.float32))
    assert np.array_equal(unpack_mask(m.cpu().numpy().view(np.uint32), C), m_ref)
