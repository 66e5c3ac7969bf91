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


def run_prefill(total, as_benched=False):
    """``as_benched``: the launch configuration bench.py times: the input vouched for as not written by
    the previous call (each chunk arrives in a buffer of its own), no mask, the state carried in
    place -- 4096-token calls then take the single-wave form that runs its gate pass before it
    waits for the previous call."""
    import torch
    from paper_2604_04250_b200 import binding as cb
    cfg = inputs.CONFIGS[2]
    flags = cb.CAWN_FLAG_INPUT_INDEPENDENT if as_benched else 0
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
        prm = cb.make_params(cfg.B, n, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=flags)
        d_p = torch.from_numpy(p).cuda()
        cb.cawn_phase_accumulate_fwd(prm, d_p, d_g, d_t, y[:, :n], ws, state_in=state, state_out=state,
                                     gate_mask=None if as_benched else mask[:, :n])
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


def test_config2_two_million_tokens_as_benched():
    """The same 2,000,000-token stream in the launch configuration the bench times (calls overlap:
    each fetches its chunk and runs its gate pass while the one before it drains)."""
    y, s, _, y_ref, s_ref, _, ncalls = run_prefill(inputs.CONFIGS[2].L, as_benched=True)
    assert ncalls == 489 and y.shape[1] == 1152
    assert floored_rel_err(y, y_ref, axes=(0, 1)) < 1e-3
    assert floored_rel_err(s, s_ref) < 1e-3


def test_prefill_as_benched_every_chunk():
    """A shorter stream in the benched configuration, every chunk's outputs against the oracle."""
    import torch
    from paper_2604_04250_b200 import binding as cb
    cfg = inputs.CONFIGS[2]
    C, chunk, nchunks = cfg.C, cfg.chunk, 12
    stream = inputs.prefill_stream(cfg, total=nchunks * chunk)
    gamma, theta = next(stream)
    chunks = list(stream)
    d_g, d_t = torch.from_numpy(gamma).cuda(), torch.from_numpy(theta).cuda()
    d_ps = [torch.from_numpy(p).cuda() for p in chunks]
    ys = [torch.full((cfg.B, chunk, C), float("nan"), dtype=torch.complex64, device="cuda") for _ in chunks]
    prm = cb.make_params(cfg.B, chunk, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=cb.CAWN_FLAG_INPUT_INDEPENDENT)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    state = torch.zeros((cfg.B, C), dtype=torch.complex64, device="cuda")
    for d_p, y in zip(d_ps, ys):                      # issued back to back, no synchronisation in between
        cb.cawn_phase_accumulate_fwd(prm, d_p, d_g, d_t, y, ws, state_in=state, state_out=state)
    assert cb.cawn_poll_status(ws) == 0
    y_ref, s_ref, _ = oracle.forward(np.concatenate(chunks, axis=1), gamma, theta, cfg.gate_eps)
    got = np.concatenate([y.cpu().numpy() for y in ys], axis=1)
    assert floored_rel_err(got, y_ref, axes=(0, 1)) < 1e-4
    assert floored_rel_err(state.cpu().numpy(), s_ref) < 1e-4
