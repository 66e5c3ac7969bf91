"""Helpers for the GPU parity tests: run the C-ABI entry points on numpy inputs."""
import numpy as np
import torch

from paper_2604_04250_b200 import binding as cb


def dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_fwd(p, gamma, theta, gate_eps, state_in=None, clamp_abs=0.0, want_mask=True,
            in_place=False, H=None):
    """Cartesian forward through cawn_phase_accumulate_fwd.  Returns numpy (y, state_out, mask_words)."""
    B, L, C = p.shape
    H = H or 1
    prm = cb.make_params(B, L, H, C // H, gate_eps=gate_eps, clamp_abs=clamp_abs)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    d_p, d_g, d_t, d_si = dev(p), dev(gamma), dev(theta), dev(state_in)
    d_y = d_p if in_place else torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda")
    d_so = torch.full((B, C), float("nan"), dtype=torch.complex64, device="cuda")
    MW = (C + 31) // 32
    d_m = torch.zeros((B, L, MW), dtype=torch.int32, device="cuda") if want_mask else None
    cb.cawn_phase_accumulate_fwd(prm, d_p, d_g, d_t, d_y, ws, state_in=d_si, state_out=d_so,
                                 gate_mask=d_m)
    st = cb.cawn_poll_status(ws)
    assert st == 0, cb.status_string(st)
    mask = d_m.cpu().numpy().view(np.uint32) if want_mask else None
    return d_y.cpu().numpy(), d_so.cpu().numpy(), mask
