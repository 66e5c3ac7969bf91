"""GPU parity: chunked prefill with O(1) state passing (config 2): 2,000,000 tokens fed in calls of
4096 (488 full chunks and one of 1,152), B=1, C=768.  The oracle walks the same stream once,
sequentially, in fp64 (its own state carried in double between the chunks it is fed, which is the
same sequence of operations as one uninterrupted pass).  Compared: the final carried state and the
last chunk's outputs within 1e-3, gate masks of the last chunk exactly."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err, unpack_mask


def run_prefill(total):
    import torch
    from paper_2604_04250_b200 import binding as cb
    cfg = inputs.CONFIGS[2]
    C, chunk = cfg.C, cfg.chunk
    stream = inputs.prefill_stream(cfg, total=total)
    gamma, theta = next(stream)
    d_g, d_t = torch.from_numpy(gamma).cuda(), torch.from_numpy(theta).cuda()
    prm_full = cb.make_params(cfg.B, chunk, cfg.H, cfg.F, gate_eps=cfg.gate_eps)
    ws = cb.new_workspace(prm_full, cb.CAWN_OP_FWD)          # one workspace serves every call
    state = torch.zeros((cfg.B, C), dtype=torch.complex64, device="cuda")
    y = torch.empty((cfg.B, chunk, C), dtype=torch.complex64, device="cuda")
    mask = torch.zeros((cfg.B, chunk, C // 32), dtype=torch.int32, device="cuda")
    state64 = np.zeros((cfg.B, C), np.complex128)
    ncalls = 0
    for p in stream:
        n = p.shape[1]
        prm = cb.make_params(cfg.B, n, cfg.H, cfg.F, gate_eps=cfg.gate_eps)
        d_p = torch.from_numpy(p).cuda()
        cb.cawn_phase_accumulate_fwd(prm, d_p, d_g, d_t, y[:, :n], ws, state_in=state, state_out=state,
                                     gate_mask=mask[:, :n])
        y_ref, state64, m_ref = oracle.forward(p, gamma, theta, cfg.gate_eps, state_in=state64)
        ncalls += 1
    assert cb.cawn_poll_status(ws) == 0
    return (y[:, :n].cpu().numpy(), state.cpu().numpy(), mask[:, :n].cpu().numpy().view(np.uint32),
            y_ref, state64, m_ref, ncalls)


def test_prefill_short_stream_ragged_tail():
    y, s, m, y_ref, s_ref, m_ref, ncalls = run_prefill(3 * 4096 + 1152)
    assert ncalls == 4
    assert floored_rel_err(y, y_ref, axes=(0, 1)) < 1e-4
    assert floored_rel_err(s, s_ref) < 1e-4
    assert np.array_equal(unpack_mask(m, 768), m_ref)


def test_config2_two_million_tokens():
    y, s, m, y_ref, s_ref, m_ref, ncalls = run_prefill(inputs.CONFIGS[2].L)
    assert ncalls == 489 and y.shape[1] == 1152
    assert floored_rel_err(y, y_ref, axes=(0, 1)) < 1e-3
    assert floored_rel_err(s, s_ref) < 1e-3
    assert np.array_equal(unpack_mask(m, 768), m_ref)
