"""The allocation-free forward entry point, cawn_phase_accumulate_fwd_static.

Some users of this library are handed input and output buffers and nothing else: a plugin in a
serving process whose device memory all belongs to one pool, or a callback that must not touch
the allocator.  They cannot bring the carry workspace the ordinary forward needs, so the library
carries a fixed 4 MiB scratch array of its own for them.  These tests call that entry point
through the C ABI twice in a row (the array keeps whatever the previous call left behind) and
compare with the ordinary entry point on the same inputs and with the CPU oracle, check the
status word it hands back (an Inf input must show up there, and the call after it must be clean
again), the zero-length call, and that what it cannot do is refused before anything runs.
Collected last on purpose.
"""
import ctypes

import numpy as np
import pytest

import oracle
from paper_2604_04250_b200 import binding as cb, inputs
from helpers import floored_rel_err, unpack_mask

TOL = 1e-4


def test_too_large_is_refused_on_the_host():
    import __graft_entry__ as entry
    entry.build()
    big = cb.make_params(64, 1 << 16, 12, 64)
    assert cb.cawn_workspace_bytes(big, cb.CAWN_OP_FWD) > cb.CAWN_STATIC_SCRATCH_BYTES
    a = 0x10000   # never dereferenced: the size check comes first
    rc = cb.lib().cawn_phase_accumulate_fwd_static(ctypes.byref(big), a, a, a, None, a, None, None, None, None)
    assert rc == cb.CAWN_ERR_STATIC_TOO_LARGE
    assert "scratch" in cb.status_string(rc)


def test_fused_and_dynamic_requests_are_refused_on_the_host():
    import __graft_entry__ as entry
    entry.build()
    a = 0x10000   # never dereferenced: these checks come before anything touches a pointer
    for prm in (cb.make_params(2, 256, 1, 64, conv_k=4), cb.make_params(2, 256, 1, 64, flags=cb.CAWN_FLAG_RETENTION_DYNAMIC)):
        rc = cb.lib().cawn_phase_accumulate_fwd_static(ctypes.byref(prm), a, a, a, None, a, None, None, None, None)
        assert rc == cb.CAWN_ERR_UNSUPPORTED
    # a missing array is reported as such, before anything is put on a stream
    prm = cb.make_params(2, 256, 1, 64)
    rc = cb.lib().cawn_phase_accumulate_fwd_static(ctypes.byref(prm), a, None, a, None, a, None, None, None, None)
    assert rc == cb.CAWN_ERR_NULL_POINTER


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_twice():
    import torch
    from gpu_util import dev
    # two different problems back to back: the second finds the first one's records in the array
    for seed, (B, L, C) in ((31, (4, 2048, 256)), (32, (3, 1500, 192))):
        d = inputs.scan_inputs(B, L, C, seed=seed, with_state=True)
        prm = cb.make_params(B, L, 1, C, gate_eps=0.1)
        p, g, t, si = dev(d["p"]), dev(d["gamma"]), dev(d["theta"]), dev(d["state_in"])
        MW = (C + 31) // 32

        ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
        y_ref = torch.empty_like(p)
        so_ref = torch.empty_like(si)
        m_ref = torch.zeros((B, L, MW), dtype=torch.int32, device="cuda")
        cb.cawn_phase_accumulate_fwd(prm, p, g, t, y_ref, ws, state_in=si, state_out=so_ref, gate_mask=m_ref)
        assert cb.cawn_poll_status(ws) == 0

        y = torch.full_like(p, float("nan"))
        so = torch.full_like(si, float("nan"))
        m = torch.zeros((B, L, MW), dtype=torch.int32, device="cuda")
        status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
        cb.cawn_phase_accumulate_fwd_static(prm, p, g, t, y, state_in=si, state_out=so, gate_mask=m,
                                            device_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert floored_rel_err(y.cpu().numpy(), y_ref.cpu().numpy().astype(np.complex128), axes=(0, 1)) < TOL
        assert floored_rel_err(so.cpu().numpy(), so_ref.cpu().numpy().astype(np.complex128)) < TOL
        assert torch.equal(m, m_ref)
        # same kernel, same launch shape, same combine order: the two entry points agree bit for bit
        assert torch.equal(y.view(torch.float32).view(torch.int32), y_ref.view(torch.float32).view(torch.int32))


def _static_call(d, B, L, C, clamp_abs=0.0):
    import torch
    from gpu_util import dev
    prm = cb.make_params(B, L, 1, C, gate_eps=0.1, clamp_abs=clamp_abs)
    p, si = dev(d["p"]), dev(d["state_in"])
    y = torch.full_like(p, float("nan"))
    so = torch.full_like(si, float("nan"))
    m = torch.zeros((B, L, (C + 31) // 32), dtype=torch.int32, device="cuda")
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    cb.cawn_phase_accumulate_fwd_static(prm, p, dev(d["gamma"]), dev(d["theta"]), y, state_in=si, state_out=so,
                                        gate_mask=m, device_status=status)
    torch.cuda.synchronize()
    return y.cpu().numpy(), so.cpu().numpy(), m.cpu().numpy().view(np.uint32), int(status.item())


@pytest.mark.gpu
def test_static_scratch_against_the_oracle_ragged_shape():
    """Odd channel count (no 16-byte rows), a length that is not a multiple of the 128-step tile, a
    carried state, the output clamp, and the gate mask, against the fp64 oracle."""
    B, L, C = 3, 1000 + 37, 77
    d = inputs.scan_inputs(B, L, C, seed=33, with_state=True)
    y, so, mw, status = _static_call(d, B, L, C, clamp_abs=3.0)
    y_ref, so_ref, m_ref = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1, clamp_abs=3.0,
                                          state_in=d["state_in"].astype(np.complex128))
    assert status == 0
    assert floored_rel_err(y, y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so, so_ref) < TOL
    assert np.array_equal(unpack_mask(mw, C), m_ref)


@pytest.mark.gpu
def test_static_scratch_reports_nonfinite_and_recovers():
    """An Inf among the pushes reaches the chain's last state: the status word handed back carries
    CAWN_STATUS_NONFINITE.  The next call on the shared array starts from a clean status."""
    B, L, C = 2, 600, 64
    d = inputs.scan_inputs(B, L, C, seed=34, with_state=True)
    bad = {k: (v.copy() if hasattr(v, "copy") else v) for k, v in d.items()}
    bad["p"][1, 300, 5] = np.complex64(complex(np.inf, 0.0))
    _, _, _, status = _static_call(bad, B, L, C)
    assert status == cb.CAWN_STATUS_NONFINITE
    y, so, _, status = _static_call(d, B, L, C)
    assert status == 0
    y_ref, so_ref, _ = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1, state_in=d["state_in"].astype(np.complex128))
    assert floored_rel_err(y, y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so, so_ref) < TOL


@pytest.mark.gpu
def test_static_scratch_zero_length_passes_the_state_through():
    import torch
    from gpu_util import dev
    B, C = 2, 96
    d = inputs.scan_inputs(B, 4, C, seed=35, with_state=True)
    prm = cb.make_params(B, 0, 1, C, gate_eps=0.1)
    si = dev(d["state_in"])
    so = torch.full_like(si, float("nan"))
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    cb.cawn_phase_accumulate_fwd_static(prm, None, dev(d["gamma"]), dev(d["theta"]), None, state_in=si, state_out=so,
                                        device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(so.view(torch.float32), si.view(torch.float32))
