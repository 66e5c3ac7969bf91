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
