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


def state_blob(B, C, conv_k, P=None, tail=None):
    """Device state blob: P [B,C] complex64, then (16-byte aligned) the conv history [B,conv_k-1,C] float."""
    prm = cb.make_params(B, 1, 1, C, conv_k=conv_k)
    n = cb.cawn_workspace_bytes(prm, cb.CAWN_OP_STATE)
    buf = np.zeros(n, np.uint8)
    off = (B * C * 8 + 15) // 16 * 16
    if P is not None:
        buf[:B * C * 8] = np.ascontiguousarray(P, dtype=np.complex64).view(np.uint8).ravel()
    if tail is not None and conv_k > 1:
        buf[off:off + B * (conv_k - 1) * C * 4] = np.ascontiguousarray(tail, dtype=np.float32).view(np.uint8).ravel()
    return torch.from_numpy(buf).cuda(), off


def split_blob(blob, off, B, C, conv_k):
    raw = blob.cpu().numpy()
    P = raw[:B * C * 8].view(np.complex64).reshape(B, C)
    tail = raw[off:off + B * (conv_k - 1) * C * 4].view(np.float32).reshape(B, conv_k - 1, C)
    return P, tail


def run_fused(h, w, gamma, theta, gate_eps, gate_tau, bias=None, clamp_silu=False, P_in=None,
              tail_in=None, clamp_abs=0.0, H=None):
    """Fused mixing path through cawn_phase_accumulate_fwd.  Returns numpy (y, P_out, tail_out, mask_words)."""
    B, L, C = h.shape
    Kc = w.shape[1]
    H = H or 1
    flags = cb.CAWN_FLAG_PRELUDE_CLAMP_SILU if clamp_silu else 0
    prm = cb.make_params(B, L, H, C // H, gate_eps=gate_eps, gate_tau=float(gate_tau), clamp_abs=clamp_abs,
                         conv_k=Kc, flags=flags)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    have_state = P_in is not None or tail_in is not None
    s_in, off = state_blob(B, C, Kc, P_in, tail_in)
    s_out, _ = state_blob(B, C, Kc)
    s_out.fill_(0xFF)
    d_y = torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda")
    MW = (C + 31) // 32
    d_m = torch.zeros((B, L, MW), dtype=torch.int32, device="cuda")
    cb.cawn_phase_accumulate_fwd(prm, dev(h), dev(gamma), dev(theta), d_y, ws, conv_w=dev(w),
                                 conv_bias=dev(bias), state_in=s_in if have_state else None,
                                 state_out=s_out, gate_mask=d_m)
    st = cb.cawn_poll_status(ws)
    assert st == 0, cb.status_string(st)
    P_out, tail_out = split_blob(s_out, off, B, C, Kc)
    return d_y.cpu().numpy(), P_out, tail_out, d_m.cpu().numpy().view(np.uint32)
