"""Pins for the oracle's gate and forward recurrence against things that are not the oracle:
closed forms, a library IIR filter, brute-force O(L^2) sums, invariants and hand-made ties."""
import math
import os

import numpy as np
import pytest
import scipy.signal

import oracle
from paper_2604_04250_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def brute_force(z, gamma, theta, state_in=None):
    """P_t = a^(t+1) S_in + sum_{s<=t} a^(t-s) z_s with a^n from pow/cos/sin: no recurrence."""
    B, L, C = z.shape
    g = gamma.astype(np.float64)
    th = theta.astype(np.float64)
    n = np.arange(L + 1, dtype=np.float64)[:, None]
    apow = (g[None, :] ** n) * (np.cos(n * th[None, :]) + 1j * np.sin(n * th[None, :]))  # [L+1, C]
    out = np.zeros((B, L, C), np.complex128)
    for t in range(L):
        w = apow[t::-1][:t + 1]            # a^(t-s) for s = 0..t
        out[:, t, :] = np.einsum("sc,bsc->bc", w, z[:, :t + 1, :])
        if state_in is not None:
            out[:, t, :] += apow[t + 1] * state_in
    return out


def test_geometric_series_constant_input():
    # constant z, constant a  =>  P_t = z (1 - a^(t+1)) / (1 - a)
    L, C = 300, 5
    gamma = np.array([0.9, 0.99, 0.5, 0.999, 0.95], np.float32)
    theta = np.array([0.0, 0.05, 1.0, 0.1, 2.5], np.float32)
    z0 = np.array([1.0 + 0j, 0.3 - 0.7j, -1j, 0.25 + 0.25j, -0.5 + 0.1j])
    z = np.broadcast_to(z0, (1, L, C)).copy()
    y, so = oracle.scan(z, theta, gamma=gamma)
    a = gamma.astype(np.float64) * np.exp(1j * theta.astype(np.float64))
    t = np.arange(L)[:, None]
    want = z0 * (1 - a ** (t + 1)) / (1 - a)
    np.testing.assert_allclose(y[0], want, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(so[0], want[-1], rtol=1e-12, atol=1e-13)


def test_unit_retention_zero_rotation_is_prefix_sum():
    rng = np.random.default_rng(5)
    z = rng.normal(size=(2, 100, 3)) + 1j * rng.normal(size=(2, 100, 3))
    y, so = oracle.scan(z, np.zeros(3, np.float32), gamma=np.ones(3, np.float32))
    np.testing.assert_allclose(y, np.cumsum(z, axis=1), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(so, z.sum(axis=1), rtol=1e-13, atol=1e-13)


def test_impulse_response_phase_advances_by_distance_times_theta():
    # An impulse m e^{i phi} injected at tau is seen at t as m gamma^(t-tau) e^{i(phi+(t-tau)theta)}.
    L, tau = 64, 9
    gamma = np.array([0.97, 0.8], np.float32)
    theta = np.array([0.3, 0.011], np.float32)
    m, phi = 0.7, 1.1
    z = np.zeros((1, L, 2), np.complex128)
    z[0, tau, :] = m * np.exp(1j * phi)
    y, _ = oracle.scan(z, theta, gamma=gamma)
    assert np.all(y[0, :tau] == 0)
    d = np.arange(L - tau)[:, None]
    want = m * gamma.astype(np.float64) ** d * np.exp(1j * (phi + d * theta.astype(np.float64)))
    np.testing.assert_allclose(y[0, tau:], want, rtol=1e-12, atol=1e-14)
    # the sign of the rotation: a positive theta turns the phasor counter-clockwise
    assert np.angle(y[0, tau + 1, 0] / y[0, tau, 0]) == pytest.approx(float(theta[0]), rel=1e-6)


def test_matches_library_iir_filter():
    # y_t = z_t + a y_{t-1} is the one-pole IIR filter 1 / (1 - a q^-1)
    d = inputs.scan_inputs(2, 500, 6, seed=11)
    z, _ = oracle.gate(d["p"], 0.0)
    y, _ = oracle.scan(z, d["theta"], gamma=d["gamma"])
    a = d["gamma"].astype(np.float64) * np.exp(1j * d["theta"].astype(np.float64))
    for j in range(6):
        want = scipy.signal.lfilter([1.0], [1.0, -a[j]], z[:, :, j], axis=1)
        np.testing.assert_allclose(y[:, :, j], want, rtol=1e-11, atol=1e-12)


def test_config0_against_brute_force():
    cfg = inputs.CONFIGS[0]
    d = inputs.config_inputs(cfg, with_state=True)
    z, mask = oracle.gate(d["p"], cfg.gate_eps)
    for si in (None, d["state_in"].astype(np.complex128)):
        y, so = oracle.scan(z, d["theta"], gamma=d["gamma"], state_in=si)
        want = brute_force(z, d["gamma"], d["theta"], si)
        np.testing.assert_allclose(y, want, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(so, want[:, -1], rtol=1e-11, atol=1e-12)
    # the gate really does something on this config (|p| ~ U[0,1), eps = 0.1)
    assert 0.05 < 1.0 - mask.mean() < 0.15


def test_brute_force_small_with_paper_theta():
    C = 8
    rng = np.random.default_rng(3)
    z = rng.normal(size=(2, 40, C)) + 1j * rng.normal(size=(2, 40, C))
    gamma = rng.uniform(0.3, 1.0, C).astype(np.float32)
    theta = inputs.paper_theta(C)
    si = rng.normal(size=(2, C)) + 1j * rng.normal(size=(2, C))
    y, so = oracle.scan(z, theta, gamma=gamma, state_in=si)
    np.testing.assert_allclose(y, brute_force(z, gamma, theta, si), rtol=1e-12, atol=1e-12)


def test_paper_theta_golden():
    # theta_j = 10000^(-2j/(HK)): values fixed by the formula for HK = 256
    rows = [l.split() for l in open(os.path.join(GOLDEN, "theta_paper_hk256.txt"))
            if l.strip() and not l.startswith("#")]
    th = inputs.paper_theta(256)
    for j, v in rows:
        assert th[int(j)] == pytest.approx(float(v), rel=1e-6)


def test_linearity_without_gate():
    rng = np.random.default_rng(8)
    z1 = rng.normal(size=(1, 50, 4)) + 1j * rng.normal(size=(1, 50, 4))
    z2 = rng.normal(size=(1, 50, 4)) + 1j * rng.normal(size=(1, 50, 4))
    gamma = rng.uniform(0.5, 1, 4).astype(np.float32)
    theta = rng.uniform(0, 1, 4).astype(np.float32)
    al, be = 0.7 - 0.2j, -1.3 + 0.4j
    y1, _ = oracle.scan(z1, theta, gamma=gamma)
    y2, _ = oracle.scan(z2, theta, gamma=gamma)
    y12, _ = oracle.scan(al * z1 + be * z2, theta, gamma=gamma)
    np.testing.assert_allclose(y12, al * y1 + be * y2, rtol=1e-12, atol=1e-12)


def test_magnitude_bound():
    d = inputs.scan_inputs(1, 200, 8, seed=2)
    z, _ = oracle.gate(d["p"], 0.1)
    y, _ = oracle.scan(z, d["theta"], gamma=d["gamma"])
    zeros = np.zeros(8, np.float32)
    bound, _ = oracle.scan(np.abs(z).astype(np.complex128), zeros, gamma=d["gamma"])
    assert np.all(np.abs(y) <= bound.real * (1 + 1e-12) + 1e-15)


# ---------------------------------------------------------------- gate
def test_gate_threshold_above_every_magnitude_gives_decayed_state():
    d = inputs.scan_inputs(2, 30, 4, seed=4, with_state=True)
    si = d["state_in"].astype(np.complex128)
    y, so, mask = oracle.forward(d["p"], d["gamma"], d["theta"], gate_eps=1.5, state_in=si)
    assert mask.sum() == 0
    a = d["gamma"].astype(np.float64) * np.exp(1j * d["theta"].astype(np.float64))
    np.testing.assert_allclose(so, a ** 30 * si, rtol=1e-12)
    y0, so0, _ = oracle.forward(d["p"], d["gamma"], d["theta"], gate_eps=1.5)
    assert np.all(y0 == 0) and np.all(so0 == 0)


def test_gate_zero_threshold_is_always_open():
    d = inputs.scan_inputs(1, 20, 4, seed=6)
    d["p"][0, 3, 1] = 0.0
    z, mask = oracle.gate(d["p"], 0.0)
    assert mask.all()
    assert np.array_equal(z, d["p"].astype(np.complex128))


def test_gate_ties_pass_and_one_ulp_below_fails():
    eps = np.float32(0.1)
    below = np.nextafter(eps, np.float32(0))
    above = np.nextafter(eps, np.float32(1))
    p = np.array([eps, below, above, -eps, 0.0], np.float32).astype(np.complex64)
    pi = (1j * p).astype(np.complex64)
    for arr in (p, pi):
        z, mask = oracle.gate(arr, float(eps))
        assert mask.tolist() == [1, 0, 1, 1, 0]
        assert np.array_equal(z, np.where(mask, arr, 0).astype(np.complex128))
    # 3-4-5 triangle scaled so that |p| = eps up to fp32 rounding of the legs
    q = np.array([np.float32(0.06) + 1j * np.float32(0.08)], np.complex64)
    s = float(np.float64(q.real[0]) ** 2 + np.float64(q.imag[0]) ** 2)
    _, mask = oracle.gate(q, float(eps))
    assert mask[0] == (s >= float(np.float64(eps) ** 2))


def test_gate_is_select_not_multiply():
    p = np.array([np.inf + 0j, np.nan + 0j, 1e-30 + 0j], np.complex64)
    z, mask = oracle.gate(p, 0.1)
    assert mask.tolist() == [1, 0, 0]
    assert z[1] == 0 and z[2] == 0


# ---------------------------------------------------------------- state passing
@pytest.mark.parametrize("splits", [[256], [1, 255], [100, 0, 56, 100], [255, 1], [64] * 4,
                                    [7, 13, 1, 1, 200, 34]])
def test_chunked_equals_unchunked(splits):
    cfg = inputs.CONFIGS[0]
    d = inputs.config_inputs(cfg)
    y_full, so_full, m_full = oracle.forward(d["p"], d["gamma"], d["theta"], cfg.gate_eps)
    state, t0 = None, 0
    for n in splits:
        y, state, m = oracle.forward(d["p"][:, t0:t0 + n], d["gamma"], d["theta"],
                                     cfg.gate_eps, state_in=state)
        # same sequence of double operations => bit-equal, not just close
        assert np.array_equal(y, y_full[:, t0:t0 + n])
        assert np.array_equal(m, m_full[:, t0:t0 + n])
        t0 += n
    assert t0 == cfg.L and np.array_equal(state, so_full)


def test_empty_call_returns_state_unchanged():
    si = np.array([[1 + 2j, -3 + 0.5j]])
    y, so = oracle.scan(np.zeros((1, 0, 2), np.complex128), np.array([0.1, 0.2], np.float32),
                        gamma=np.array([0.9, 0.8], np.float32), state_in=si)
    assert y.shape == (1, 0, 2) and np.array_equal(so, si)


# ---------------------------------------------------------------- clamp
def test_clamp_is_output_only():
    L, C = 400, 3
    z = np.ones((1, L, C), np.complex128) * (1 + 1j)
    gamma = np.array([0.9999, 0.99, 0.5], np.float32)
    theta = np.zeros(C, np.float32)
    y_raw, so_raw = oracle.scan(z, theta, gamma=gamma)
    y, so = oracle.scan(z, theta, gamma=gamma, clamp_abs=100.0)
    assert np.abs(y_raw.real).max() > 100.0          # the clamp does trigger
    assert np.abs(y.real).max() <= 100.0 and np.abs(y.imag).max() <= 100.0
    want = np.clip(y_raw.real, -100, 100) + 1j * np.clip(y_raw.imag, -100, 100)
    assert np.array_equal(y, want)
    assert np.array_equal(so, so_raw)                # the carried state is not clamped


# ---------------------------------------------------------------- dynamic retention
def test_dynamic_retention_constant_logit_equals_static():
    B, L, H, F = 2, 60, 3, 4
    rng = np.random.default_rng(9)
    z = rng.normal(size=(B, L, H * F)) + 1j * rng.normal(size=(B, L, H * F))
    theta = rng.uniform(0, 0.5, H * F).astype(np.float32)
    head_logit = np.array([0.5, 2.0, -1.0], np.float32)
    fb = np.linspace(3, 0, F).astype(np.float32)
    gl = np.broadcast_to(head_logit, (B, L, H)).copy()
    s = head_logit.astype(np.float64)[:, None] + fb.astype(np.float64)[None, :]
    gamma64 = (1 / (1 + np.exp(-s))).reshape(-1)
    gamma = gamma64.astype(np.float32)               # static path takes fp32 gamma
    y_dyn, so_dyn = oracle.scan(z, theta, gamma_logit=gl, freq_bias=fb)
    y_st, so_st = oracle.scan(z, theta, gamma=gamma, H=H)
    # differ only by the fp32 rounding of gamma (~6e-8 per step)
    np.testing.assert_allclose(y_dyn, y_st, rtol=0, atol=2e-4 * np.abs(y_st).max())
    # and against the closed form with the unrounded gamma
    a = gamma64 * np.exp(1j * theta.astype(np.float64))
    want = np.zeros_like(z)
    P = np.zeros((B, H * F), np.complex128)
    for t in range(L):
        P = z[:, t] + a * P
        want[:, t] = P
    np.testing.assert_allclose(y_dyn, want, rtol=1e-11, atol=1e-12)


def test_dynamic_retention_against_brute_force_products():
    B, L, H, F = 1, 24, 2, 3
    C = H * F
    rng = np.random.default_rng(10)
    z = rng.normal(size=(B, L, C)) + 1j * rng.normal(size=(B, L, C))
    theta = rng.uniform(0, 1, C).astype(np.float32)
    dyn = inputs.dynamic_retention_inputs(B, L, H, F, seed=10)
    y, _ = oracle.scan(z, theta, **dyn)
    s = dyn["gamma_logit"].astype(np.float64)[..., None] + dyn["freq_bias"].astype(np.float64)
    g = (1 / (1 + np.exp(-s))).reshape(B, L, C)       # j = h*F + k
    th = theta.astype(np.float64)
    want = np.zeros_like(z)
    for t in range(L):
        for s_ in range(t + 1):
            # z_s is decayed by gamma_{s+1} ... gamma_t and rotated (t - s) times
            w = np.prod(g[:, s_ + 1:t + 1], axis=1) * np.exp(1j * (t - s_) * th)
            want[:, t] += w * z[:, s_]
    np.testing.assert_allclose(y, want, rtol=1e-11, atol=1e-12)
