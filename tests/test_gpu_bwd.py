"""GPU parity: the reverse-scan backward through the C ABI against the fp64 oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err

TOL = 1e-4


def run_bwd(d, eps, saved_kind, use_state=True, grad_clamp_abs=0.0, want_param=True, in_place=False):
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    B, L, C = d["p"].shape
    prm = cb.make_params(B, L, 1, C, gate_eps=eps, grad_clamp_abs=grad_clamp_abs)
    si = d["state_in"] if use_state else None
    gso = d["grad_state_out"] if use_state else None
    g, t = dev(d["gamma"]), dev(d["theta"])
    if saved_kind == cb.CAWN_SAVED_STATES:
        # the forward's own unclamped output is what a training step would have saved
        y = torch.empty((B, L, C), dtype=torch.complex64, device="cuda")
        wf = cb.new_workspace(prm, cb.CAWN_OP_FWD)
        cb.cawn_phase_accumulate_fwd(prm, dev(d["p"]), g, t, y, wf, state_in=dev(si))
        assert cb.cawn_poll_status(wf) == 0
        saved, op = y, cb.CAWN_OP_BWD_SAVED
    else:
        saved, op = dev(d["p"]), cb.CAWN_OP_BWD_PUSHES
    ws = cb.new_workspace(prm, op)
    gy = dev(d["grad_y"])
    gp = gy if in_place else torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda")
    gg = torch.full((C,), float("nan"), device="cuda") if want_param else None
    gt = torch.full((C,), float("nan"), device="cuda") if want_param else None
    gsi = torch.full((B, C), float("nan"), dtype=torch.complex64, device="cuda")
    cb.cawn_phase_accumulate_bwd(prm, saved, saved_kind, g, t, gy, gp, ws, state_in=dev(si),
                                 grad_state_out=dev(gso), grad_gamma=gg, grad_theta=gt,
                                 grad_state_in=gsi)
    assert cb.cawn_poll_status(ws) == 0
    out = {"dp": gp.cpu().numpy(), "dstate_in": gsi.cpu().numpy()}
    if want_param:
        out["dgamma"] = gg.cpu().numpy()
        out["dtheta"] = gt.cpu().numpy()
    return out


def reference(d, eps, use_state=True, grad_clamp_abs=0.0):
    z, _ = oracle.gate(d["p"], eps)
    si = d["state_in"].astype(np.complex128) if use_state else None
    gso = d["grad_state_out"].astype(np.complex128) if use_state else None
    return oracle.scan_bwd(z, d["theta"], d["grad_y"], gamma=d["gamma"], state_in=si,
                           dstate_out=gso, grad_clamp_abs=grad_clamp_abs)


def compare(got, ref, L, tol=TOL):
    if L:
        assert floored_rel_err(got["dp"], ref["dp"], axes=(0, 1)) < tol
    assert floored_rel_err(got["dstate_in"], ref["dstate_in"]) < tol
    for k in ("dgamma", "dtheta"):
        if k in got:
            assert not np.isnan(got[k]).any()
            assert floored_rel_err(got[k], ref[k]) < tol, k


@pytest.mark.parametrize("saved_kind", [0, 1])
@pytest.mark.parametrize("B,L,C", [(1, 1, 64), (2, 5, 64), (1, 64, 64), (2, 65, 128), (2, 300, 64),
                                   (1, 1000, 192), (2, 333, 100), (1, 2049, 768)])
def test_bwd_shapes(B, L, C, saved_kind):
    d = inputs.scan_inputs(B, L, C, seed=200 + L + C, with_state=True, with_grad=True)
    compare(run_bwd(d, 0.1, saved_kind), reference(d, 0.1), L)


def test_bwd_config3():
    cfg = inputs.CONFIGS[3]
    d = inputs.config_inputs(cfg)
    got = run_bwd(d, cfg.gate_eps, 0, use_state=False)
    compare(got, reference(d, cfg.gate_eps, use_state=False), cfg.L)


def test_bwd_without_parameter_gradients_and_in_place():
    d = inputs.scan_inputs(2, 500, 128, seed=21, with_state=True, with_grad=True)
    got = run_bwd(d, 0.1, 0, want_param=False, in_place=True)
    compare(got, reference(d, 0.1), 500)


def test_bwd_gradient_clamp():
    d = inputs.scan_inputs(2, 400, 64, seed=22, with_state=True, with_grad=True)
    d["grad_y"] = (d["grad_y"] * 40).astype(np.complex64)
    got = run_bwd(d, 0.1, 0, grad_clamp_abs=100.0)
    ref = reference(d, 0.1, grad_clamp_abs=100.0)
    assert np.abs(got["dp"].real).max() == 100.0
    assert floored_rel_err(got["dp"], ref["dp"], axes=(0, 1)) < TOL
    assert np.abs(got["dgamma"]).max() <= 100.0
    assert np.allclose(got["dgamma"], ref["dgamma"], rtol=1e-3, atol=1e-2)


def test_bwd_repeatable_bitwise():
    d = inputs.scan_inputs(2, 1500, 128, seed=23, with_state=True, with_grad=True)
    a = run_bwd(d, 0.1, 0)
    b = run_bwd(d, 0.1, 0)
    for k in a:
        assert np.array_equal(a[k].view(np.uint32), b[k].view(np.uint32)), k
