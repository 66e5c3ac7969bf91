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


def test_bf16_refused_where_not_built():
    import torch
    from paper_2604_04250_b200 import binding as cb
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
