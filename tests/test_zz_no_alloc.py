"""The allocation-free forward entry point, cawn_phase_accumulate_fwd_static.

Some users of this library are handed input and output buffers and nothing else: a plugin in a
serving process whose device memory all belongs to one pool, or a callback that must not touch
the allocator.  They cannot bring the carry workspace the ordinary forward needs, so the library
carries a fixed 4 MiB scratch array of its own for them.  These tests call that entry point
through the C ABI twice in a row (the array keeps whatever the previous call left behind) and
compare with the ordinary entry point on the same inputs, and check that a problem too large for
the array is refused before anything runs.  Collected last on purpose.
"""
import ctypes

import numpy as np
import pytest

from paper_2604_04250_b200 import binding as cb, inputs
from helpers import floored_rel_err

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
