"""GPU: device-side status reporting.  A carry wait that runs into its bound (made to, by the
wait hook: one tile keeps its summary to itself) ends the kernel with CAWN_ERR_CARRY_TIMEOUT instead
of hanging, leaves the workspace usable, and the next call is correct again; Inf in the input
raises CAWN_STATUS_NONFINITE; NaN pushes are gated away silently."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err


def _setup(B, L, C, seed):
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    d = inputs.scan_inputs(B, L, C, seed)
    prm = cb.make_params(B, L, 1, C, gate_eps=0.1)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    y = torch.full((B, L, C), float("nan"), dtype=torch.complex64, device="cuda")
    return d, prm, ws, y, dev, cb


def test_withheld_tile_times_out_and_the_workspace_recovers():
    B, L, C = 2, 2048, 64                        # 16 tiles of 128 steps per chain
    d, prm, ws, y, dev, cb = _setup(B, L, C, 31)
    p, g, t = dev(d["p"]), dev(d["gamma"]), dev(d["theta"])
    ref, _, _ = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1)
    cb.cawn_workspace_set_wait_hook(ws, 3, 2000)
    cb.cawn_phase_accumulate_fwd(prm, p, g, t, y, ws)
    st = cb.cawn_poll_status(ws)
    assert st & cb.CAWN_ERR_CARRY_TIMEOUT, st
    got = y.cpu().numpy()
    # tiles 0..3 do not depend on the silent tile's summary: their rows are complete and right
    assert floored_rel_err(got[:, :512], ref[:, :512]) < 1e-4
    assert cb.cawn_poll_status(ws) == 0           # the record was cleared by the poll
    # hook off: the same workspace gives the full, correct result
    cb.cawn_workspace_set_wait_hook(ws, -1, 0)
    y.fill_(float("nan"))
    cb.cawn_phase_accumulate_fwd(prm, p, g, t, y, ws)
    assert cb.cawn_poll_status(ws) == 0
    assert floored_rel_err(y.cpu().numpy(), ref) < 1e-4


def test_timeout_in_the_backward():
    import torch
    B, L, C = 1, 1024, 64                        # 16 tiles of 64 steps
    d, prm, _, _, dev, cb = _setup(B, L, C, 32)
    rng = np.random.default_rng(3)
    G = (rng.normal(size=(B, L, C)) + 1j * rng.normal(size=(B, L, C))).astype(np.complex64)
    ws = cb.new_workspace(prm, cb.CAWN_OP_BWD_SAVED)
    gp = torch.zeros((B, L, C), dtype=torch.complex64, device="cuda")
    P = dev(d["p"])                               # any array serves as the saved states here
    cb.cawn_workspace_set_wait_hook(ws, 0, 1500)
    cb.cawn_phase_accumulate_bwd(prm, P, cb.CAWN_SAVED_STATES, dev(d["gamma"]), dev(d["theta"]), dev(G), gp, ws)
    assert cb.cawn_poll_status(ws) & cb.CAWN_ERR_CARRY_TIMEOUT
    cb.cawn_workspace_set_wait_hook(ws, -1, 0)
    cb.cawn_phase_accumulate_bwd(prm, P, cb.CAWN_SAVED_STATES, dev(d["gamma"]), dev(d["theta"]), dev(G), gp, ws)
    assert cb.cawn_poll_status(ws) == 0
    ref = oracle.scan_bwd(np.zeros((B, L, C), np.complex128), d["theta"], G, gamma=d["gamma"])
    assert floored_rel_err(gp.cpu().numpy(), ref["dp"]) < 1e-4


def test_inf_input_raises_nonfinite_and_nan_push_is_gated_away():
    B, L, C = 1, 600, 64
    d, prm, ws, y, dev, cb = _setup(B, L, C, 33)
    p = d["p"].copy()
    p[0, 300, 5] = np.nan + 0j                    # fails |p| >= eps: dropped like a closed gate
    cb.cawn_phase_accumulate_fwd(prm, dev(p), dev(d["gamma"]), dev(d["theta"]), y, ws)
    assert cb.cawn_poll_status(ws) == 0
    q = d["p"].copy(); q[0, 300, 5] = 0
    ref, _, _ = oracle.forward(q, d["gamma"], d["theta"], 0.1)
    assert floored_rel_err(y.cpu().numpy(), ref) < 1e-4
    p[0, 300, 5] = np.inf
    cb.cawn_phase_accumulate_fwd(prm, dev(p), dev(d["gamma"]), dev(d["theta"]), y, ws)
    assert cb.cawn_poll_status(ws) == cb.CAWN_STATUS_NONFINITE
    got = y.cpu().numpy()
    assert not np.isfinite(got[0, 300:, 5]).all() and np.isfinite(got[0, :300]).all()
    # a non-finite carried state is reported too
    s_in = np.zeros((B, C), np.complex64); s_in[0, 7] = np.inf
    cb.cawn_phase_accumulate_fwd(prm, dev(d["p"]), dev(d["gamma"]), dev(d["theta"]), y, ws, state_in=dev(s_in))
    assert cb.cawn_poll_status(ws) == cb.CAWN_STATUS_NONFINITE


def test_hook_argument_checks():
    import torch
    from paper_2604_04250_b200 import binding as cb
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    for tile, bound in ((70000, 10), (1, 70000)):
        with pytest.raises(cb.CawnError) as e:
            cb.cawn_workspace_set_wait_hook(ws, tile, bound)
        assert e.value.status == cb.CAWN_ERR_INVALID_ARG
