"""GPU parity: the Cartesian forward (gate, scan, clamp, state passing) through the C ABI
against the fp64 oracle on the same seeded inputs.  Tolerances: floored relative error 1e-4 on
outputs and carried state (1e-3 after the 2M-token prefill), gate masks bit-exact."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err, unpack_mask

TOL = 1e-4


def check_fwd(d, eps, state_in=None, clamp_abs=0.0, tol=TOL, in_place=False, H=None):
    from gpu_util import run_fwd
    p = d["p"]
    B, L, C = p.shape
    si64 = None if state_in is None else state_in.astype(np.complex128)
    y_ref, so_ref, m_ref = oracle.forward(p, d["gamma"], d["theta"], eps, state_in=si64,
                                          clamp_abs=clamp_abs)
    y, so, mw = run_fwd(p.copy(), d["gamma"], d["theta"], eps, state_in=state_in,
                        clamp_abs=clamp_abs, in_place=in_place, H=H)
    assert np.array_equal(unpack_mask(mw, C), m_ref), "gate mask differs"
    assert not np.isnan(y.view(np.float32)).any()
    if L:
        assert floored_rel_err(y, y_ref, axes=(0, 1)) < tol
    assert floored_rel_err(so, so_ref) < tol
    return y, so


def test_config0_tiny():
    cfg = inputs.CONFIGS[0]
    check_fwd(inputs.config_inputs(cfg), cfg.gate_eps, H=cfg.H)


def test_config1_training_shape():
    cfg = inputs.CONFIGS[1]
    check_fwd(inputs.config_inputs(cfg), cfg.gate_eps, H=cfg.H)


@pytest.mark.parametrize("B,L,C", [
    (1, 1, 64), (2, 3, 64), (1, 16, 64), (1, 17, 64), (3, 32, 128), (1, 33, 64),
    (2, 127, 64), (2, 128, 64), (2, 129, 192), (1, 1000, 64), (2, 515, 768),
    (1, 300, 48), (2, 200, 100), (1, 130, 1), (1, 140, 33), (1, 4097, 128),
])
def test_ragged_shapes_with_state(B, L, C):
    d = inputs.scan_inputs(B, L, C, seed=100 + L + C, with_state=True)
    check_fwd(d, 0.1, state_in=d["state_in"])


def test_long_single_call_many_tiles():
    # 1024 tiles along time in one call: the look-back chain is far longer than what is resident
    d = inputs.scan_inputs(1, 131072 + 5, 64, seed=7, with_state=True)
    check_fwd(d, 0.1, state_in=d["state_in"])


def test_high_retention_long_memory():
    # gamma pinned at the top of the range: the case where a rounded multiplier would drift
    d = inputs.scan_inputs(2, 8192, 64, seed=8, gamma_lo=0.9999, gamma_hi=0.99999)
    check_fwd(d, 0.1)


def test_paper_theta_and_zero_gate():
    d = inputs.scan_inputs(2, 700, 256, seed=9)
    d["theta"] = inputs.paper_theta(256)
    check_fwd(d, 0.0)


def test_gate_above_every_magnitude():
    from gpu_util import run_fwd
    d = inputs.scan_inputs(2, 300, 64, seed=10, with_state=True)
    y, so, mw = run_fwd(d["p"], d["gamma"], d["theta"], 1.5, state_in=d["state_in"])
    assert not mw.any()
    a = d["gamma"].astype(np.float64) * np.exp(1j * d["theta"].astype(np.float64))
    assert floored_rel_err(so, a ** 300 * d["state_in"].astype(np.complex128)) < TOL
    y0, so0, _ = run_fwd(d["p"], d["gamma"], d["theta"], 1.5)
    assert not y0.any() and not so0.any()


def test_gate_ties_are_exact():
    from gpu_util import run_fwd
    eps = np.float32(0.1)
    vals = np.array([eps, np.nextafter(eps, np.float32(0)), np.nextafter(eps, np.float32(1)),
                     -eps, 0.0, 0.06], np.float32)
    p = np.zeros((1, 6, 64), np.complex64)
    p.real[0, :, :] = vals[:, None]
    p.imag[0, 5, :] = np.float32(0.08)
    g = np.full(64, 0.5, np.float32)
    t = np.zeros(64, np.float32)
    _, _, m_ref = oracle.forward(p, g, t, float(eps))
    _, _, mw = run_fwd(p, g, t, float(eps))
    assert np.array_equal(unpack_mask(mw, 64), m_ref)
    assert m_ref[0, :5, 0].tolist() == [1, 0, 1, 1, 0]


def test_clamp_is_output_only():
    d = inputs.scan_inputs(2, 3000, 64, seed=11, gamma_lo=0.9995, gamma_hi=0.9999)
    d["p"] = (d["p"] * 8).astype(np.complex64)
    y, so = check_fwd(d, 0.1, clamp_abs=100.0)
    assert np.abs(y.real).max() == 100.0 and np.abs(y.imag).max() <= 100.0
    assert np.abs(so).max() > 100.0


def test_in_place():
    d = inputs.scan_inputs(2, 400, 128, seed=12)
    check_fwd(d, 0.1, in_place=True)


@pytest.mark.parametrize("splits", [[300, 212], [1, 127, 128, 256], [5, 0, 507], [128] * 4])
def test_chunked_state_passing(splits):
    from gpu_util import run_fwd
    d = inputs.scan_inputs(2, 512, 128, seed=13)
    y_ref, so_ref, _ = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1)
    state, t0 = None, 0
    for n in splits:
        y, state, _ = run_fwd(d["p"][:, t0:t0 + n].copy(), d["gamma"], d["theta"], 0.1, state_in=state)
        if n:
            assert floored_rel_err(y, y_ref[:, t0:t0 + n], axes=(0, 1)) < TOL
        t0 += n
    assert floored_rel_err(state, so_ref) < TOL


def test_state_carry_entry_point():
    import torch
    from gpu_util import dev, run_fwd
    from paper_2604_04250_b200 import binding as cb
    d = inputs.scan_inputs(2, 1000, 128, seed=14, with_state=True)
    # the definition: run the segment from S_prev
    _, so_ref, _ = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1,
                                  state_in=d["state_in"].astype(np.complex128))
    _, local, _ = run_fwd(d["p"], d["gamma"], d["theta"], 0.1)          # from a zero state
    prm = cb.make_params(2, 1000, 1, 128)
    out = torch.empty((2, 128), dtype=torch.complex64, device="cuda")
    cb.cawn_state_carry(prm, dev(d["state_in"]), dev(local), 1000, dev(d["gamma"]), dev(d["theta"]), out)
    assert floored_rel_err(out.cpu().numpy(), so_ref) < TOL
    # a very long gap: a^n from pow/sincos, compared with the closed form (retention close
    # enough to 1 that a^n does not underflow)
    n = 1_500_000
    gam = inputs.log_uniform(np.random.default_rng(5), 0.99999, 0.999999, 128).astype(np.float32)
    cb.cawn_state_carry(prm, dev(d["state_in"]), dev(np.zeros_like(local)), n, dev(gam),
                        dev(d["theta"]), out)
    a_n = gam.astype(np.float64) ** n * np.exp(1j * n * d["theta"].astype(np.float64))
    assert floored_rel_err(out.cpu().numpy(), a_n * d["state_in"].astype(np.complex128)) < TOL


def test_host_buffer_entry_point():
    import torch
    from paper_2604_04250_b200 import binding as cb
    d = inputs.scan_inputs(2, 333, 128, seed=15, with_state=True)
    B, L, C = d["p"].shape
    prm = cb.make_params(B, L, 1, C, gate_eps=0.1)
    scratch = cb.new_workspace(prm, cb.CAWN_OP_FWD_HOST)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    p, g, t, si = pin(d["p"]), pin(d["gamma"]), pin(d["theta"]), pin(d["state_in"])
    y = torch.empty((B, L, C), dtype=torch.complex64).pin_memory()
    so = torch.empty((B, C), dtype=torch.complex64).pin_memory()
    m = torch.zeros((B, L, C // 32), dtype=torch.int32).pin_memory()
    cb.cawn_phase_accumulate_fwd_host(prm, p, g, t, y, scratch, state_in_host=si,
                                      state_out_host=so, gate_mask_host=m)
    torch.cuda.synchronize()
    y_ref, so_ref, m_ref = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1,
                                          state_in=d["state_in"].astype(np.complex128))
    assert floored_rel_err(y.numpy(), y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so.numpy(), so_ref) < TOL
    assert np.array_equal(unpack_mask(m.numpy().view(np.uint32), C), m_ref)


@pytest.mark.parametrize("B,L,C", [(4, 4096, 128), (11, 2048, 64), (1, 20000, 128), (1, 9000, 192), (2, 16500, 128), (8, 4100, 256)])
def test_host_buffer_entry_point_sliced(B, L, C):
    """Calls of 8 MB and more go through the two copy streams in slices: batch rows for B >= 2,
    stretches of time with the state carried for B = 1.  Two calls in a row reuse the pipes."""
    import torch
    from paper_2604_04250_b200 import binding as cb
    d = inputs.scan_inputs(B, L, C, seed=150 + B, with_state=True)
    prm = cb.make_params(B, L, 1, C, gate_eps=0.1)
    scratch = cb.new_workspace(prm, cb.CAWN_OP_FWD_HOST)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    p, g, t, si = pin(d["p"]), pin(d["gamma"]), pin(d["theta"]), pin(d["state_in"])
    y_ref, so_ref, m_ref = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1,
                                          state_in=d["state_in"].astype(np.complex128))
    for _ in range(2):
        y = torch.full((B, L, C), float("nan"), dtype=torch.complex64).pin_memory()
        so = torch.full((B, C), float("nan"), dtype=torch.complex64).pin_memory()
        m = torch.zeros((B, L, C // 32), dtype=torch.int32).pin_memory()
        cb.cawn_phase_accumulate_fwd_host(prm, p, g, t, y, scratch, state_in_host=si,
                                          state_out_host=so, gate_mask_host=m)
        torch.cuda.current_stream().synchronize()        # the caller's stream alone: the call joined its pipes into it
        assert floored_rel_err(y.numpy(), y_ref, axes=(0, 1)) < TOL
        assert floored_rel_err(so.numpy(), so_ref) < TOL
        assert np.array_equal(unpack_mask(m.numpy().view(np.uint32), C), m_ref)


@pytest.mark.parametrize("B,L,C", [(1, 1153, 64), (1, 1920, 128), (2, 2048, 64), (1, 2049, 192), (1, 4096, 768), (3, 3000, 100),
                                   (1, 8 * 128 + 1, 64), (1, 16 * 128, 64), (1, 17 * 128 + 5, 64), (1, 31 * 128, 64)])
def test_lengths_around_checkpoint_tiles(B, L, C):
    """Lengths on both sides of one, two and four checkpoint tiles (every seventh tile of 128 steps
    publishes its carry-in), with a carried state and no mask; twice, bit for bit."""
    from gpu_util import run_fwd
    d = inputs.scan_inputs(B, L, C, seed=170 + L % 97, with_state=True)
    y, so, _ = run_fwd(d["p"], d["gamma"], d["theta"], 0.1, state_in=d["state_in"], want_mask=False)
    y_ref, so_ref, _ = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1, state_in=d["state_in"].astype(np.complex128))
    assert floored_rel_err(y, y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(so, so_ref) < TOL
    y2, so2, _ = run_fwd(d["p"], d["gamma"], d["theta"], 0.1, state_in=d["state_in"], want_mask=False)
    assert np.array_equal(y.view(np.uint32), y2.view(np.uint32)) and np.array_equal(so.view(np.uint32), so2.view(np.uint32))


def test_repeatable_bitwise():
    from gpu_util import run_fwd
    d = inputs.scan_inputs(4, 2048, 256, seed=16)
    y1, s1, m1 = run_fwd(d["p"], d["gamma"], d["theta"], 0.1)
    y2, s2, m2 = run_fwd(d["p"], d["gamma"], d["theta"], 0.1)
    assert np.array_equal(y1.view(np.uint32), y2.view(np.uint32))
    assert np.array_equal(s1.view(np.uint32), s2.view(np.uint32)) and np.array_equal(m1, m2)


def test_workspace_reuse_across_calls_and_shapes():
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    big = cb.make_params(2, 2048, 1, 128, gate_eps=0.1)
    ws = cb.new_workspace(big, cb.CAWN_OP_FWD)
    for seed, L in ((1, 2048), (2, 130), (3, 2048), (4, 1), (5, 1999)):
        d = inputs.scan_inputs(2, L, 128, seed=seed)
        prm = cb.make_params(2, L, 1, 128, gate_eps=0.1)
        y = torch.empty((2, L, 128), dtype=torch.complex64, device="cuda")
        cb.cawn_phase_accumulate_fwd(prm, dev(d["p"]), dev(d["gamma"]), dev(d["theta"]), y, ws)
        assert cb.cawn_poll_status(ws) == 0
        y_ref, _, _ = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1)
        assert floored_rel_err(y.cpu().numpy(), y_ref, axes=(0, 1)) < TOL


def test_unsupported_and_error_paths_on_device_memory():
    import torch
    from paper_2604_04250_b200 import binding as cb
    prm = cb.make_params(1, 64, 1, 64)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    x = torch.zeros((1, 64, 64), dtype=torch.complex64, device="cuda")
    g = torch.ones(64, device="cuda")
    with pytest.raises(cb.CawnError) as e:
        cb.cawn_phase_accumulate_fwd(prm, x, g, g, x, ws[:128])
    assert e.value.status == cb.CAWN_ERR_WORKSPACE_TOO_SMALL
    assert cb.cawn_poll_status(ws) == 0


def test_overlapped_calls_match_serial_calls_bitwise():
    # CAWN_FLAG_INPUT_INDEPENDENT lets a call fetch its input while the previous call on the stream
    # drains; states and workspace are still only touched after it.  A chain of calls passing the
    # state along must give bit-identical results with and without the flag.
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    B, L, C, n = 2, 1024, 256, 6
    ds = [inputs.scan_inputs(B, L, C, seed=60 + i) for i in range(n)]
    g, t = dev(ds[0]["gamma"]), dev(ds[0]["theta"])
    ps = [dev(d["p"]) for d in ds]
    outs = []
    for flags in (0, cb.CAWN_FLAG_INPUT_INDEPENDENT):
        prm = cb.make_params(B, L, 1, C, gate_eps=0.1, flags=flags)
        ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
        state = torch.zeros((B, C), dtype=torch.complex64, device="cuda")
        ys = [torch.empty((B, L, C), dtype=torch.complex64, device="cuda") for _ in range(n)]
        for i in range(n):
            cb.cawn_phase_accumulate_fwd(prm, ps[i], g, t, ys[i], ws, state_in=state, state_out=state)
        assert cb.cawn_poll_status(ws) == 0
        outs.append((torch.stack(ys).cpu().numpy(), state.cpu().numpy()))
    assert np.array_equal(outs[0][0].view(np.uint32), outs[1][0].view(np.uint32))
    assert np.array_equal(outs[0][1].view(np.uint32), outs[1][1].view(np.uint32))
    # and the chain equals one long oracle pass
    p_all = np.concatenate([d["p"] for d in ds], axis=1)
    y_ref, so_ref, _ = oracle.forward(p_all, ds[0]["gamma"], ds[0]["theta"], 0.1)
    assert floored_rel_err(np.concatenate(list(outs[1][0]), axis=1), y_ref, axes=(0, 1)) < TOL
    assert floored_rel_err(outs[1][1], so_ref) < TOL


def test_config1_as_benched_rotating_buffers():
    """Config 1 in the launch configuration bench.py times: the input vouched for, no mask, state out,
    steps issued back to back over rotating buffer sets with no synchronisation in between.  Every
    step's output against the oracle (the sets are time-rolled copies of one draw, as in the bench)."""
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    cfg = inputs.CONFIGS[1]
    d = inputs.config_inputs(cfg)
    B, L, C, nsets, nsteps = cfg.B, cfg.L, cfg.C, 3, 7
    p0 = dev(d["p"])
    ps = [torch.roll(p0, shifts=17 * i, dims=1).contiguous() for i in range(nsets)]
    ys = [torch.full_like(p0, float("nan")) for _ in range(nsteps)]
    g, t = dev(d["gamma"]), dev(d["theta"])
    prm = cb.make_params(B, L, cfg.H, cfg.F, gate_eps=cfg.gate_eps, flags=cb.CAWN_FLAG_INPUT_INDEPENDENT)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    state = torch.empty((B, C), dtype=torch.complex64, device="cuda")
    for i in range(nsteps):
        cb.cawn_phase_accumulate_fwd(prm, ps[i % nsets], g, t, ys[i], ws, state_out=state)
    assert cb.cawn_poll_status(ws) == 0
    refs = [oracle.forward(np.roll(d["p"], 17 * i, axis=1), d["gamma"], d["theta"], cfg.gate_eps) for i in range(nsets)]
    for i in range(nsteps):
        assert floored_rel_err(ys[i].cpu().numpy(), refs[i % nsets][0], axes=(0, 1)) < TOL, i
    assert floored_rel_err(state.cpu().numpy(), refs[(nsteps - 1) % nsets][1]) < TOL
