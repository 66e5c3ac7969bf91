"""GPU parity: the fused Resonance mixing path (causal depthwise conv prelude, phasor map, gate,
push, scan) through the C ABI against the fp64 oracle.  Masks exact, values within 1e-4."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err, unpack_mask

TOL = 1e-4


def check_fused(d, eps, clamp_silu=False, P_in=None, clamp_abs=0.0, H=None):
    from gpu_util import run_fused
    h, w = d["h"], d["conv_w"]
    B, L, C = h.shape
    tau = inputs.gate_tau(eps)
    bias, tail = d.get("conv_bias"), d.get("tail_in")
    P64 = None if P_in is None else P_in.astype(np.complex128)
    y_ref, so_ref, m_ref, tail_ref = oracle.fused_forward(h, w, d["gamma"], d["theta"], eps, tau, bias=bias,
                                                          clamp_silu=clamp_silu, tail_in=tail, state_in=P64,
                                                          clamp_abs=clamp_abs)
    y, so, tail_out, mw = run_fused(h, w, d["gamma"], d["theta"], eps, tau, bias=bias, clamp_silu=clamp_silu,
                                    P_in=P_in, tail_in=tail, clamp_abs=clamp_abs, H=H)
    assert np.array_equal(unpack_mask(mw, C), m_ref), "gate mask differs"
    if L:
        assert not np.isnan(y.view(np.float32)).any()
        assert floored_rel_err(y, y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so, so_ref) < TOL
    if w.shape[1] > 1:
        assert np.array_equal(tail_out, tail_ref)
    return y, m_ref


@pytest.mark.parametrize("B,L,C,Kc", [
    (1, 1, 64, 4), (2, 2, 64, 4), (1, 3, 64, 3), (2, 17, 64, 4), (1, 128, 64, 4), (2, 129, 128, 3),
    (2, 300, 192, 4), (1, 1000, 64, 2), (2, 257, 100, 4), (1, 140, 33, 4), (1, 200, 64, 1), (1, 515, 768, 4),
])
def test_fused_shapes(B, L, C, Kc):
    d = inputs.fused_inputs(B, L, C, seed=300 + L + C, conv_k=Kc, with_tail=Kc > 1, with_bias=True)
    rng = np.random.default_rng(L)
    P_in = (rng.normal(0, 2, (B, C)) + 1j * rng.normal(0, 2, (B, C))).astype(np.complex64)
    check_fused(d, 0.1, P_in=P_in)


def taps_at_8_byte_offset(monkeypatch):
    """Make gpu_util.dev place every [C, 4] float array 8 bytes past a 16-byte boundary: the library
    asks 8-byte alignment of the taps, and its 16-byte tap loads have to stand aside then."""
    import torch
    import gpu_util
    real = gpu_util.dev

    def dev8(a):
        t = real(a)
        if t is not None and t.ndim == 2 and t.shape[1] == 4 and t.dtype == torch.float32:
            big = torch.empty(t.numel() + 2, dtype=t.dtype, device=t.device)
            v = big[2:].view(t.shape)
            v.copy_(t)
            assert v.data_ptr() % 16 == 8
            return v
        return t
    monkeypatch.setattr(gpu_util, "dev", dev8)


def test_fused_taps_only_8_byte_aligned(monkeypatch):
    taps_at_8_byte_offset(monkeypatch)
    d = inputs.fused_inputs(2, 300, 192, seed=77, conv_k=4, with_tail=True, with_bias=True)
    check_fused(d, 0.1)


def test_fused_gate_closes_some_and_zero_state():
    d = inputs.fused_inputs(2, 2048, 128, seed=41)
    _, m_ref = check_fused(d, 0.1)
    frac = 1.0 - m_ref.mean()
    assert 0.001 < frac < 0.2            # the 0.1 gate does close on part of the N(0, ...) conv outputs


def test_fused_clamp_silu_all_open():
    d = inputs.fused_inputs(2, 700, 128, seed=42, with_tail=True, with_bias=True)
    d["h"] = (d["h"] * 30).astype(np.float32)          # drives the conv output past the +-50 clamp
    _, m_ref = check_fused(d, 0.1, clamp_silu=True)
    assert m_ref.all()


def test_fused_output_clamp_and_zero_gate():
    d = inputs.fused_inputs(1, 3000, 64, seed=43, gamma_lo=0.9995, gamma_hi=0.9999)
    check_fused(d, 0.0, clamp_abs=5.0)


@pytest.mark.parametrize("splits", [[300, 212], [1, 2, 1, 508], [130, 0, 382], [2, 510]])
def test_fused_chunked_state_and_history_passing(splits):
    from gpu_util import run_fused
    d = inputs.fused_inputs(2, 512, 128, seed=44, with_bias=True)
    tau = inputs.gate_tau(0.1)
    y_ref, so_ref, _, tail_ref = oracle.fused_forward(d["h"], d["conv_w"], d["gamma"], d["theta"], 0.1, tau,
                                                      bias=d["conv_bias"])
    P, tail, t0 = None, None, 0
    for n in splits:
        y, P, tail, _ = run_fused(d["h"][:, t0:t0 + n].copy(), d["conv_w"], d["gamma"], d["theta"], 0.1, tau,
                                  bias=d["conv_bias"], P_in=P, tail_in=tail)
        P, tail = P.copy(), tail.copy()
        if n:
            assert floored_rel_err(y, y_ref[:, t0:t0 + n], axes=(0, 1)) < TOL
        t0 += n
    assert floored_rel_err(P, so_ref) < TOL
    assert np.array_equal(tail, tail_ref)


def test_fused_config4_full_size():
    """Config 4 at full size (B=16, L=8192, C=768) in the launch configuration the bench times:
    outputs, gate masks, carried state and conv history of all sixteen batch rows against the
    oracle, which walks the rows one by one (about two seconds each)."""
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    cfg = inputs.CONFIGS[4]
    d = inputs.config_inputs(cfg)
    B, L, C = cfg.B, cfg.L, cfg.C
    tau = inputs.gate_tau(cfg.gate_eps)
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, gate_tau=float(tau), conv_k=cfg.conv_k,
                         flags=cb.CAWN_FLAG_INPUT_INDEPENDENT)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    y = torch.empty((B, L, C), dtype=torch.complex64, device="cuda")
    m = torch.zeros((B, L, C // 32), dtype=torch.int32, device="cuda")
    s_out, off = state_blob(B, C, cfg.conv_k)
    s_out.fill_(0xFF)
    cb.cawn_phase_accumulate_fwd(prm, dev(d["h"]), dev(d["gamma"]), dev(d["theta"]), y, ws,
                                 conv_w=dev(d["conv_w"]), gate_mask=m, state_out=s_out)
    assert cb.cawn_poll_status(ws) == 0
    P_out, tail_out = split_blob(s_out, off, B, C, cfg.conv_k)
    worst = 0.0
    for b in range(B):
        y_ref, so_ref, m_ref, tail_ref = oracle.fused_forward(d["h"][b:b + 1], d["conv_w"], d["gamma"], d["theta"],
                                                              cfg.gate_eps, tau)
        worst = max(worst, floored_rel_err(y[b:b + 1].cpu().numpy(), y_ref, axes=(0, 1)))
        assert worst < TOL, b
        assert np.array_equal(unpack_mask(m[b:b + 1].cpu().numpy().view(np.uint32), C), m_ref), b
        assert floored_rel_err(P_out[b:b + 1], so_ref) < TOL, b
        assert np.array_equal(tail_out[b:b + 1], tail_ref), b
