"""Pins for the oracle's conv prelude / phasor map and for its reverse-scan backward."""
import math

import numpy as np
import pytest
import scipy.signal

import oracle
from paper_2604_04250_b200 import inputs


# ---------------------------------------------------------------- conv prelude
def phasor(x):
    m = 1 / (1 + np.exp(-x))
    return m * np.exp(1j * np.pi * np.tanh(x))


def test_prelude_identity_conv_is_the_phasor_map():
    rng = np.random.default_rng(0)
    h = rng.normal(size=(2, 17, 5)).astype(np.float32)
    w = np.ones((5, 1), np.float32)
    z, mask, tail = oracle.prelude(h, w)
    assert mask.all() and tail.shape == (2, 0, 5)
    np.testing.assert_allclose(z, phasor(h.astype(np.float64)), rtol=1e-13, atol=1e-15)
    # hand-checkable points: x=0 -> m=1/2, phase 0 ; large x -> m->1, phase -> pi
    z0, _, _ = oracle.prelude(np.array([[[0.0], [40.0]]], np.float32), np.ones((1, 1), np.float32))
    assert z0[0, 0, 0] == pytest.approx(0.5 + 0j)
    assert z0[0, 1, 0] == pytest.approx(-1.0 + 0j, abs=1e-12)


def test_prelude_impulse_reads_taps_back_in_order():
    # an impulse at time 5 makes u_{5+d} = w[Kc-1-d]: the LAST tap multiplies the current token
    Kc, L = 4, 12
    w = np.array([[0.1, -0.2, 0.3, 0.7]], np.float32)
    h = np.zeros((1, L, 1), np.float32)
    h[0, 5, 0] = 1.0
    z, _, _ = oracle.prelude(h, w)
    u = np.zeros(L)
    for d in range(Kc):
        u[5 + d] = w[0, Kc - 1 - d]
    np.testing.assert_allclose(z[0, :, 0], phasor(u), rtol=1e-13)


@pytest.mark.parametrize("Kc", [2, 3, 4])
def test_prelude_equals_textbook_causal_fir(Kc):
    d = inputs.fused_inputs(2, 50, 6, seed=21, conv_k=Kc, with_bias=True)
    z, _, _ = oracle.prelude(d["h"], d["conv_w"], d["conv_bias"])
    for c in range(6):
        taps = d["conv_w"][c, ::-1].astype(np.float64)     # FIR coefficient of delay d is w[Kc-1-d]
        u = scipy.signal.lfilter(taps, [1.0], d["h"][:, :, c].astype(np.float64), axis=1)
        u = u + float(d["conv_bias"][c])
        np.testing.assert_allclose(z[:, :, c], phasor(u), rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("splits", [[50], [1, 49], [2, 1, 0, 47], [25, 25], [3, 3, 44]])
def test_prelude_carried_tail_equals_unchunked(splits):
    Kc = 4
    d = inputs.fused_inputs(2, 50, 6, seed=22, conv_k=Kc)
    tau = inputs.gate_tau(0.1)
    z_full, m_full, tail_full = oracle.prelude(d["h"], d["conv_w"], gate_eps=0.1, gate_tau=tau)
    tail, t0 = None, 0
    for n in splits:
        z, m, tail = oracle.prelude(d["h"][:, t0:t0 + n], d["conv_w"], tail_in=tail,
                                    gate_eps=0.1, gate_tau=tau)
        assert np.array_equal(z, z_full[:, t0:t0 + n])
        assert np.array_equal(m, m_full[:, t0:t0 + n])
        t0 += n
    assert np.array_equal(tail, tail_full)
    assert np.array_equal(tail_full, d["h"][:, -(Kc - 1):])


def test_prelude_gate_threshold_on_conv_output():
    # m >= eps  <=>  u >= logit(eps); closed gates give exact zeros
    d = inputs.fused_inputs(1, 400, 8, seed=23, conv_k=4)
    eps = 0.1
    tau = inputs.gate_tau(eps)
    assert float(tau) == pytest.approx(math.log(eps / (1 - eps)), rel=1e-6)
    z, mask, _ = oracle.prelude(d["h"], d["conv_w"], gate_eps=eps, gate_tau=tau)
    z_open, _, _ = oracle.prelude(d["h"], d["conv_w"])
    closed = mask == 0
    assert 0.002 < closed.mean() < 0.05            # P(u < -2.197), u ~ N(0, 1) here: about 1.4 %
    assert np.all(z[closed] == 0) and np.array_equal(z[~closed], z_open[~closed])
    m = np.abs(z_open)
    # away from the threshold the fp32 decision agrees with the fp64 magnitude
    far = np.abs(m - eps) > 1e-5
    assert np.array_equal((m >= eps)[far], mask.astype(bool)[far])


def test_prelude_clamp_silu_keeps_every_gate_open():
    d = inputs.fused_inputs(1, 200, 8, seed=24, conv_k=3)
    d["h"][0, 10, 0] = 1e4                         # exercises the +-50 clamp
    z, mask, _ = oracle.prelude(d["h"], d["conv_w"], clamp_silu=True, gate_eps=0.1,
                                gate_tau=inputs.gate_tau(0.1))
    assert mask.all()
    assert np.abs(z).min() >= 0.43                 # sigmoid(min SiLU) = sigmoid(-0.2785)
    z1, _, _ = oracle.prelude(d["h"], d["conv_w"])
    with np.errstate(divide="ignore"):
        u = np.log(np.abs(z1) / (1 - np.abs(z1)))  # recover u from m = sigmoid(u) where safe
    ok = np.abs(u) < 20
    uc = np.clip(u, -50, 50)
    x = uc / (1 + np.exp(-uc))
    np.testing.assert_allclose(np.abs(z)[ok], (1 / (1 + np.exp(-x)))[ok], rtol=1e-9)


# ---------------------------------------------------------------- backward
def setup_bwd(B=2, L=40, C=6, seed=31, eps=0.1):
    d = inputs.scan_inputs(B, L, C, seed, gamma_lo=0.6, gamma_hi=0.99, theta_hi=0.8,
                           with_state=True, with_grad=True)
    z, _ = oracle.gate(d["p"], eps)
    return d, z


def loss(z, gamma, theta, si, G, dso, **kw):
    y, so = oracle.scan(z, theta, gamma=gamma, state_in=si, **kw)
    return float(np.sum((np.conj(G) * y).real) + np.sum((np.conj(dso) * so).real))


def test_bwd_adjoint_identity():
    d, z = setup_bwd()
    si = d["state_in"].astype(np.complex128)
    G = d["grad_y"]
    dso = d["grad_state_out"].astype(np.complex128)
    y, so = oracle.scan(z, d["theta"], gamma=d["gamma"], state_in=si)
    g = oracle.scan_bwd(z, d["theta"], G, gamma=d["gamma"], state_in=si, dstate_out=dso)
    lhs = np.sum((np.conj(G.astype(np.complex128)) * y).real) + np.sum((np.conj(dso) * so).real)
    rhs = np.sum((np.conj(g["dp"]) * z).real) + np.sum((np.conj(g["dstate_in"]) * si).real)
    assert lhs == pytest.approx(rhs, rel=1e-12)


def test_bwd_push_gradient_against_brute_force():
    d, z = setup_bwd()
    G = d["grad_y"].astype(np.complex128)
    dso = d["grad_state_out"].astype(np.complex128)
    g = oracle.scan_bwd(z, d["theta"], d["grad_y"], gamma=d["gamma"], dstate_out=dso)
    B, L, C = z.shape
    ac = d["gamma"].astype(np.float64) * np.exp(-1j * d["theta"].astype(np.float64))   # conj(a)
    Gp = G.copy()
    Gp[:, -1] += dso
    want = np.zeros_like(G)
    for t in range(L):
        for s in range(t, L):
            want[:, t] += ac ** (s - t) * Gp[:, s]
    np.testing.assert_allclose(g["dp"], want, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(g["dstate_in"], ac * want[:, 0], rtol=1e-11, atol=1e-12)


def test_bwd_push_gradient_ignores_gate_and_forward_values():
    d, z = setup_bwd()
    g1 = oracle.scan_bwd(z, d["theta"], d["grad_y"], gamma=d["gamma"])
    z_open, _ = oracle.gate(d["p"], 0.0)
    g2 = oracle.scan_bwd(z_open * 3.0, d["theta"], d["grad_y"], gamma=d["gamma"])
    assert np.array_equal(g1["dp"], g2["dp"])        # straight-through: identity at every position


def test_bwd_parameter_gradients_by_finite_differences():
    d, z = setup_bwd()
    si = d["state_in"].astype(np.complex128)
    G = d["grad_y"].astype(np.complex128)
    dso = d["grad_state_out"].astype(np.complex128)
    # fp32-representable parameters with fp32-representable perturbations
    gamma = d["gamma"]
    theta = d["theta"]
    g = oracle.scan_bwd(z, theta, d["grad_y"], gamma=gamma, state_in=si, dstate_out=dso)
    hstep = np.float32(2.0 ** -14)
    for j in range(z.shape[2]):
        for name, grad in (("gamma", g["dgamma"]), ("theta", g["dtheta"])):
            base = {"gamma": gamma.copy(), "theta": theta.copy()}
            hi = {k: v.copy() for k, v in base.items()}
            lo = {k: v.copy() for k, v in base.items()}
            hi[name][j] += hstep
            lo[name][j] -= hstep
            step = float(hi[name][j]) - float(lo[name][j])
            fd = (loss(z, hi["gamma"], hi["theta"], si, G, dso)
                  - loss(z, lo["gamma"], lo["theta"], si, G, dso)) / step
            assert grad[j] == pytest.approx(fd, rel=2e-4, abs=1e-6), (name, j)


def test_bwd_state_gradient_by_finite_differences():
    d, z = setup_bwd(B=1, L=25, C=3)
    si = d["state_in"].astype(np.complex128)
    G = d["grad_y"].astype(np.complex128)
    dso = d["grad_state_out"].astype(np.complex128)
    g = oracle.scan_bwd(z, d["theta"], d["grad_y"], gamma=d["gamma"], state_in=si, dstate_out=dso)
    h = 1e-6
    for j in range(3):
        for unit in (1.0, 1j):
            e = np.zeros_like(si)
            e[0, j] = unit * h
            fd = (loss(z, d["gamma"], d["theta"], si + e, G, dso)
                  - loss(z, d["gamma"], d["theta"], si - e, G, dso)) / (2 * h)
            got = g["dstate_in"][0, j].real if unit == 1.0 else g["dstate_in"][0, j].imag
            assert got == pytest.approx(fd, rel=1e-6, abs=1e-8)


def test_bwd_gamma_gradient_closed_form_constant_input():
    # z = 1, theta = 0, G = 1 on the last step only: Loss = sum_{s<L} gamma^s, dLoss/dgamma known
    L = 30
    gamma = np.array([0.9], np.float32)
    z = np.ones((1, L, 1), np.complex128)
    G = np.zeros((1, L, 1), np.complex64)
    G[0, -1, 0] = 1.0
    g = oracle.scan_bwd(z, np.zeros(1, np.float32), G, gamma=gamma)
    gm = float(gamma[0])
    want = sum(s * gm ** (s - 1) for s in range(1, L))
    assert g["dgamma"][0] == pytest.approx(want, rel=1e-12)
    assert g["dtheta"][0] == pytest.approx(0.0, abs=1e-12)


def test_bwd_clamp_is_pass_through_and_grad_clamp_bounds():
    d, z = setup_bwd()
    big = 50.0 * d["grad_y"]
    g = oracle.scan_bwd(z, d["theta"], big, gamma=d["gamma"])
    gc = oracle.scan_bwd(z, d["theta"], big, gamma=d["gamma"], grad_clamp_abs=100.0)
    assert np.abs(g["dp"].real).max() > 100.0
    want = np.clip(g["dp"].real, -100, 100) + 1j * np.clip(g["dp"].imag, -100, 100)
    assert np.array_equal(gc["dp"], want)
    assert np.array_equal(gc["dgamma"], np.clip(g["dgamma"], -100, 100))


def test_bwd_dynamic_retention_by_finite_differences():
    B, L, H, F = 1, 16, 2, 3
    C = H * F
    rng = np.random.default_rng(41)
    z = rng.normal(size=(B, L, C)) + 1j * rng.normal(size=(B, L, C))
    theta = rng.uniform(0, 0.8, C).astype(np.float32)
    dyn = inputs.dynamic_retention_inputs(B, L, H, F, seed=41)
    G = (rng.normal(size=(B, L, C)) + 1j * rng.normal(size=(B, L, C))).astype(np.complex64)
    si = rng.normal(size=(B, C)) + 1j * rng.normal(size=(B, C))
    g = oracle.scan_bwd(z, theta, G, state_in=si, **dyn)

    def f(gl, fb, th):
        y, _ = oracle.scan(z, th, gamma_logit=gl, freq_bias=fb, state_in=si)
        return float(np.sum((np.conj(G.astype(np.complex128)) * y).real))

    hstep = np.float32(2.0 ** -13)
    for idx in [(0, 0, 0), (0, 5, 1), (0, 15, 0), (0, 9, 1)]:
        hi, lo = dyn["gamma_logit"].copy(), dyn["gamma_logit"].copy()
        hi[idx] += hstep
        lo[idx] -= hstep
        fd = (f(hi, dyn["freq_bias"], theta) - f(lo, dyn["freq_bias"], theta)) / (float(hi[idx]) - float(lo[idx]))
        assert g["dgamma_logit"][idx] == pytest.approx(fd, rel=5e-4, abs=1e-6)
    for k in range(F):
        hi, lo = dyn["freq_bias"].copy(), dyn["freq_bias"].copy()
        hi[k] += hstep
        lo[k] -= hstep
        fd = (f(dyn["gamma_logit"], hi, theta) - f(dyn["gamma_logit"], lo, theta)) / (float(hi[k]) - float(lo[k]))
        assert g["dfreq_bias"][k] == pytest.approx(fd, rel=5e-4, abs=1e-6)
    for j in range(C):
        hi, lo = theta.copy(), theta.copy()
        hi[j] += hstep
        lo[j] -= hstep
        fd = (f(dyn["gamma_logit"], dyn["freq_bias"], hi) - f(dyn["gamma_logit"], dyn["freq_bias"], lo)) / (float(hi[j]) - float(lo[j]))
        assert g["dtheta"][j] == pytest.approx(fd, rel=5e-4, abs=1e-6)
