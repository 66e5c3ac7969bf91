"""GPU parity on seeded random shapes and option mixes, through every forward variant and the two
backwards: a net for cases the hand-picked shapes of the other files do not reach (odd channel
counts with partial groups, lengths around tile multiples, thresholds, clamps, states)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err, unpack_mask

TOL = 1e-4


def _shape(rng, max_l=700):
    B = int(rng.integers(1, 4))
    L = int(rng.choice([int(rng.integers(1, 40)), int(rng.integers(40, max_l)), 128 * int(rng.integers(1, 5)) + int(rng.integers(-2, 3))]))
    H = int(rng.integers(1, 7))
    F = int(rng.choice([1, 2, 3, 8, 16, 21, 32, 64]))
    return B, max(L, 1), H, F


@pytest.mark.parametrize("seed", range(12))
def test_random_cartesian_forward_and_backward(seed):
    import torch
    from gpu_util import dev, run_fwd
    from paper_2604_04250_b200 import binding as cb
    rng = np.random.default_rng(4000 + seed)
    B, L, H, F = _shape(rng)
    C = H * F
    eps = float(rng.choice([0.0, 0.1, 0.5]))
    clamp = float(rng.choice([0.0, 1.5]))
    d = inputs.scan_inputs(B, L, C, seed=4100 + seed, with_state=True, with_grad=True)
    use_state = bool(rng.integers(0, 2))
    si = d["state_in"] if use_state else None
    y, so, mw = run_fwd(d["p"], d["gamma"], d["theta"], eps, state_in=si, clamp_abs=clamp, H=H)
    y_ref, so_ref, m_ref = oracle.forward(d["p"], d["gamma"], d["theta"], eps, clamp_abs=clamp,
                                          state_in=None if si is None else si.astype(np.complex128))
    assert np.array_equal(unpack_mask(mw, C), m_ref)
    assert floored_rel_err(y, y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so, so_ref) < TOL
    # backward from the unclamped states
    P, _, _ = run_fwd(d["p"], d["gamma"], d["theta"], eps, state_in=si, H=H)
    prm = cb.make_params(B, L, H, F, gate_eps=eps)
    ws = cb.new_workspace(prm, cb.CAWN_OP_BWD_SAVED)
    gp = torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda")
    gg, gt = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    gsi = torch.empty((B, C), dtype=torch.complex64, device="cuda")
    cb.cawn_phase_accumulate_bwd(prm, dev(P), cb.CAWN_SAVED_STATES, dev(d["gamma"]), dev(d["theta"]), dev(d["grad_y"]), gp, ws,
                                 state_in=dev(si), grad_state_out=dev(d["grad_state_out"]), grad_gamma=gg, grad_theta=gt,
                                 grad_state_in=gsi)
    assert cb.cawn_poll_status(ws) == 0
    z, _ = oracle.gate(d["p"], eps)
    ref = oracle.scan_bwd(z, d["theta"], d["grad_y"], gamma=d["gamma"], state_in=None if si is None else si.astype(np.complex128),
                          dstate_out=d["grad_state_out"].astype(np.complex128))
    assert floored_rel_err(gp.cpu().numpy(), ref["dp"], axes=(0, 1)) < TOL
    assert floored_rel_err(gsi.cpu().numpy(), ref["dstate_in"]) < TOL
    assert floored_rel_err(gg.cpu().numpy(), ref["dgamma"]) < TOL
    assert floored_rel_err(gt.cpu().numpy(), ref["dtheta"]) < TOL


@pytest.mark.parametrize("seed", range(10))
def test_random_fused_forward_backward_and_ear(seed):
    from test_gpu_fused_bwd import make, run_mixing_bwd, reference, compare
    from test_gpu_ear import run_ear
    rng = np.random.default_rng(5000 + seed)
    B, L, H, F = _shape(rng, max_l=400)
    C = H * F
    Kc = int(rng.integers(1, 5))
    d = make(B, L, C, Kc, seed=5100 + seed, with_bias=bool(rng.integers(0, 2)))
    tail = d["gso_tail"] if Kc > 1 else None
    clamp_silu = bool(rng.integers(0, 4) == 0)
    got = run_mixing_bwd(d, 0.1, clamp_silu=clamp_silu, P_in=d["P_in"], gso_P=d["gso_P"], gso_tail=tail)
    compare(got, reference(d, 0.1, clamp_silu=clamp_silu, P_in=d["P_in"], gso_P=d["gso_P"], gso_tail=tail), L, Kc)
    if C <= 64 or 64 % F == 0:
        run_ear(B, L, H, F, int(rng.choice([1, 3])), seed=5200 + seed, fused=bool(rng.integers(0, 2)),
                clamp_abs=float(rng.choice([0.0, 2.0])))


@pytest.mark.parametrize("seed", range(8))
def test_random_bf16_and_dynamic(seed):
    from test_gpu_bf16 import run_cartesian
    from test_gpu_dynamic import make as make_dyn, run_fwd_dyn, ref_fwd
    rng = np.random.default_rng(6000 + seed)
    B, L, H, F = _shape(rng)
    C = H * F
    run_cartesian(B, L, C, 6100 + seed, bool(rng.integers(0, 2)), True, clamp_abs=float(rng.choice([0.0, 2.0])))
    d = make_dyn(B, L, H, F, seed=6200 + seed)
    _, m_ref, (y_ref, so_ref) = ref_fwd(d, 0.1)
    y, so, mw = run_fwd_dyn(d, H, F, 0.1)
    assert np.array_equal(unpack_mask(mw, C), m_ref)
    assert floored_rel_err(y.cpu().numpy(), y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so, so_ref) < TOL
