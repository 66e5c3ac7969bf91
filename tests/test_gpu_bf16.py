"""GPU parity: bfloat16 storage of the forward's input and / or output around the fp32 scan
(CAWN_FLAG_INPUT_BF16, CAWN_FLAG_OUTPUT_BF16).  The oracle is given the bf16-rounded inputs widened to
float; a bf16 output is compared within bf16's rounding (2^-8 per component: 7 stored mantissa bits) on top of the fp32
tolerance, and bit for bit against the fp32-output run rounded to bf16."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err, unpack_mask

TOL = 1e-4
TOL16 = 2.0 ** -8 + 2e-4


def _io_flags(cb, in16, out16):
    return (cb.CAWN_FLAG_INPUT_BF16 if in16 else 0) | (cb.CAWN_FLAG_OUTPUT_BF16 if out16 else 0)


def _read_y(y, out16):
    if not out16:
        return y.cpu().numpy()
    f = inputs.from_bf16(y.cpu().numpy().view(np.uint16))          # [B,L,C,2]
    return np.ascontiguousarray(f).view(np.complex64)[..., 0]


def run_cartesian(B, L, C, seed, in16, out16, clamp_abs=0.0):
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    d = inputs.scan_inputs(B, L, C, seed)
    bits, wide = inputs.to_bf16(d["p"])
    p_used = wide if in16 else d["p"]
    rng = np.random.default_rng(seed + 1)
    s_in = (rng.normal(0, 2, (B, C)) + 1j * rng.normal(0, 2, (B, C))).astype(np.complex64)
    prm = cb.make_params(B, L, 1, C, gate_eps=0.1, clamp_abs=clamp_abs, flags=_io_flags(cb, in16, out16))
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    x = torch.from_numpy(bits.view(np.int16)).cuda() if in16 else dev(d["p"])
    y = (torch.full((B, L, C, 2), -1, dtype=torch.int16, device="cuda") if out16
         else torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda"))
    so = torch.full((B, C), float("nan"), dtype=torch.complex64, device="cuda")
    m = torch.zeros((B, L, (C + 31) // 32), dtype=torch.int32, device="cuda")
    cb.cawn_phase_accumulate_fwd(prm, x, dev(d["gamma"]), dev(d["theta"]), y, ws, state_in=dev(s_in), state_out=so, gate_mask=m)
    assert cb.cawn_poll_status(ws) == 0
    ry, rso, rmask = oracle.forward(p_used, d["gamma"], d["theta"], 0.1, state_in=s_in.astype(np.complex128), clamp_abs=clamp_abs)
    got = _read_y(y, out16)
    assert not np.isnan(got.view(np.float32)).any()
    assert floored_rel_err(got, ry) < (TOL16 if out16 else TOL)
    assert floored_rel_err(so.cpu().numpy(), rso) < TOL
    assert np.array_equal(unpack_mask(m.cpu().numpy().view(np.uint32), C), rmask)
    return d, p_used, s_in, y


@pytest.mark.parametrize("in16,out16", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("B,L,C", [(1, 1, 64), (2, 20, 64), (2, 300, 128), (1, 129, 33), (2, 257, 100), (1, 515, 768)])
def test_cartesian_bf16_storage(B, L, C, in16, out16):
    run_cartesian(B, L, C, 900 + L + C, in16, out16)


def test_bf16_output_is_the_rounded_fp32_output():
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    B, L, C = 2, 700, 128
    d, p_used, s_in, y16 = run_cartesian(B, L, C, 17, True, True, clamp_abs=2.0)
    prm = cb.make_params(B, L, 1, C, gate_eps=0.1, clamp_abs=2.0)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    y32 = torch.empty((B, L, C), dtype=torch.complex64, device="cuda")
    cb.cawn_phase_accumulate_fwd(prm, dev(p_used), dev(d["gamma"]), dev(d["theta"]), y32, ws, state_in=dev(s_in))
    ref_bits, _ = inputs.to_bf16(y32.cpu().numpy())
    assert np.array_equal(y16.cpu().numpy().view(np.uint16), ref_bits)


@pytest.mark.parametrize("in16,out16", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("B,L,C,Kc", [(1, 2, 64, 4), (2, 200, 64, 4), (1, 333, 100, 3), (1, 131, 33, 4), (2, 515, 768, 4), (1, 20, 64, 2)])
def test_fused_bf16_storage(B, L, C, Kc, in16, out16):
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    d = inputs.fused_inputs(B, L, C, 950 + L, conv_k=Kc, with_tail=True)
    bits, wide = inputs.to_bf16(d["h"])
    h_used = wide if in16 else d["h"]
    eps, tau = 0.1, float(inputs.gate_tau(0.1))
    rng = np.random.default_rng(5)
    P_in = (rng.normal(0, 2, (B, C)) + 1j * rng.normal(0, 2, (B, C))).astype(np.complex64)
    prm = cb.make_params(B, L, 1, C, gate_eps=eps, gate_tau=tau, conv_k=Kc, flags=_io_flags(cb, in16, out16))
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    s_in, off = state_blob(B, C, Kc, P_in, d["tail_in"])
    s_out, _ = state_blob(B, C, Kc)
    s_out.fill_(0xFF)
    x = torch.from_numpy(bits.view(np.int16)).cuda() if in16 else dev(d["h"])
    y = (torch.full((B, L, C, 2), -1, dtype=torch.int16, device="cuda") if out16
         else torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda"))
    m = torch.zeros((B, L, (C + 31) // 32), dtype=torch.int32, device="cuda")
    cb.cawn_phase_accumulate_fwd(prm, x, dev(d["gamma"]), dev(d["theta"]), y, ws, conv_w=dev(d["conv_w"]),
                                 conv_bias=dev(d.get("conv_bias")), state_in=s_in, state_out=s_out, gate_mask=m)
    assert cb.cawn_poll_status(ws) == 0
    ry, rso, rmask, rtail = oracle.fused_forward(h_used, d["conv_w"], d["gamma"], d["theta"], eps, tau, bias=d.get("conv_bias"),
                                                 tail_in=d["tail_in"], state_in=P_in.astype(np.complex128))
    got = _read_y(y, out16)
    assert floored_rel_err(got, ry) < (TOL16 if out16 else TOL)
    P_out, tail_out = split_blob(s_out, off, B, C, Kc)
    assert floored_rel_err(P_out, rso) < TOL
    assert np.array_equal(tail_out, rtail.astype(np.float32))          # the carried history stays fp32, exact
    assert np.array_equal(unpack_mask(m.cpu().numpy().view(np.uint32), C), rmask)


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("dyn,ear", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("B,L,H,F", [(1, 2, 1, 64), (2, 200, 2, 64), (1, 333, 4, 16), (2, 515, 12, 64), (1, 131, 3, 11)])
def test_bf16_with_dynamic_retention_and_ear(B, L, H, F, dyn, ear, fused):
    """bf16 input and output around the fp32 scan in the forms of the paper's own layer: per-token
    retention and / or the Ear's convolution across the harmonics as the epilogue, Cartesian and
    fused input.  The oracle gets the widened bf16 inputs; the bf16 output is compared within its
    own rounding."""
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    C = H * F
    if ear and C > 64 and 64 % F != 0:
        pytest.skip("the Ear epilogue needs the harmonics of a head inside one 64-channel group")
    eps, tau, Kc = 0.1, float(inputs.gate_tau(0.1)), 4
    rng = np.random.default_rng(1000 + L + F)
    P_in = (rng.normal(0, 2, (B, C)) + 1j * rng.normal(0, 2, (B, C))).astype(np.complex64)
    dd = inputs.dynamic_retention_inputs(B, L, H, F, 1100 + L) if dyn else {}
    ew = rng.normal(0.0, 0.6, (2 * H, 3)).astype(np.float32)
    eb = rng.normal(0.0, 0.3, 2 * H).astype(np.float32)
    flags = _io_flags(cb, True, True) | (cb.CAWN_FLAG_RETENTION_DYNAMIC if dyn else 0)
    kw = dict(gamma_logit=dev(dd.get("gamma_logit")), freq_bias=dev(dd.get("freq_bias")))
    okw = dict(gamma_logit=dd.get("gamma_logit"), freq_bias=dd.get("freq_bias"), H=H) if dyn else {}
    if fused:
        d = inputs.fused_inputs(B, L, C, 1200 + L, conv_k=Kc, with_tail=True, with_bias=True)
        bits, wide = inputs.to_bf16(d["h"])
        y_ref, so_ref, m_ref, tail_ref = oracle.fused_forward(wide, d["conv_w"], None if dyn else d["gamma"], d["theta"], eps, tau,
                                                              bias=d["conv_bias"], tail_in=d["tail_in"],
                                                              state_in=P_in.astype(np.complex128), **okw)
        prm = cb.make_params(B, L, H, F, gate_eps=eps, gate_tau=tau, conv_k=Kc, flags=flags)
        s_in, off = state_blob(B, C, Kc, P_in, d["tail_in"])
        s_out, _ = state_blob(B, C, Kc)
        kw.update(conv_w=dev(d["conv_w"]), conv_bias=dev(d["conv_bias"]))
    else:
        d = inputs.scan_inputs(B, L, C, 1200 + L)
        bits, wide = inputs.to_bf16(d["p"])
        z, m_ref = oracle.gate(wide, eps)
        y_ref, so_ref = oracle.scan(z, d["theta"], gamma=None if dyn else d["gamma"], state_in=P_in.astype(np.complex128), **okw)
        prm = cb.make_params(B, L, H, F, gate_eps=eps, flags=flags)
        s_in = dev(P_in)
        s_out = torch.full((B, C), float("nan"), dtype=torch.complex64, device="cuda")
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    x = torch.from_numpy(bits.view(np.int16)).cuda()
    m = torch.zeros((B, L, (C + 31) // 32), dtype=torch.int32, device="cuda")
    g = None if dyn else dev(d["gamma"])
    if ear:
        zc = torch.full((B, L, 2, H, F), -1, dtype=torch.int16, device="cuda")
        cb.cawn_phase_accumulate_fwd_ear(prm, x, g, dev(d["theta"]), dev(ew), 3, zc, ws, ear_bias=dev(eb), state_in=s_in,
                                         state_out=s_out, gate_mask=m, **kw)
        got = inputs.from_bf16(zc.cpu().numpy().view(np.uint16))
        want = oracle.ear_conv(y_ref, ew, eb, H, F)
    else:
        y = torch.full((B, L, C, 2), -1, dtype=torch.int16, device="cuda")
        cb.cawn_phase_accumulate_fwd(prm, x, g, dev(d["theta"]), y, ws, state_in=s_in, state_out=s_out, gate_mask=m, **kw)
        got = _read_y(y, True)
        want = y_ref
    assert cb.cawn_poll_status(ws) == 0
    assert not np.isnan(got.view(np.float32)).any()
    assert floored_rel_err(got, want) < TOL16
    if fused:
        P_out, tail_out = split_blob(s_out, off, B, C, Kc)
        assert np.array_equal(tail_out, tail_ref.astype(np.float32))
    else:
        P_out = s_out.cpu().numpy()
    assert floored_rel_err(P_out, so_ref) < TOL                      # the carried state stays fp32
    assert np.array_equal(unpack_mask(m.cpu().numpy().view(np.uint32), C), m_ref)


def test_bf16_refused_where_not_built():
    import torch
    from paper_2604_04250_b200 import binding as cb
    # with the Ear epilogue (or time-varying retention) bf16 storage comes for input and output together
    prm = cb.make_params(1, 8, 1, 64, flags=cb.CAWN_FLAG_OUTPUT_BF16)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    x = torch.zeros((1, 8, 64), dtype=torch.complex64, device="cuda")
    g = torch.ones(64, device="cuda")
    with pytest.raises(cb.CawnError) as e:
        cb.cawn_phase_accumulate_fwd_ear(prm, x, g, g, torch.ones((2, 3), device="cuda"), 3, x.view(torch.float32), ws)
    assert e.value.status == cb.CAWN_ERR_UNSUPPORTED
    wb = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(cb.CawnError) as e:
        cb.cawn_phase_accumulate_bwd(prm, x, cb.CAWN_SAVED_STATES, g, g, x, x, wb)
    assert e.value.status == cb.CAWN_ERR_UNSUPPORTED
