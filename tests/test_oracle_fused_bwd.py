"""Pins for the oracle's backward of the fused mixing path (prelude_bwd, fused_backward) against
things that are not that code: central finite differences of the oracle's own (separately pinned)
forward, the straight-through rule stated as a projection, and chunked = unchunked."""
import numpy as np
import pytest

import oracle
from paper_2604_04250_b200 import inputs


def setup(B=2, L=24, C=5, Kc=4, seed=51, with_tail=True):
    d = inputs.fused_inputs(B, L, C, seed, conv_k=Kc, with_tail=with_tail and Kc > 1, with_bias=True)
    rng = np.random.default_rng(seed + 1)
    d["G"] = (rng.normal(size=(B, L, C)) + 1j * rng.normal(size=(B, L, C))).astype(np.complex64)
    d["state_in"] = rng.normal(size=(B, C)) + 1j * rng.normal(size=(B, C))
    d["dstate_out"] = rng.normal(size=(B, C)) + 1j * rng.normal(size=(B, C))
    return d


def loss(d, h=None, w=None, bias=None, tail=None, eps=0.0, tau=-np.inf, clamp_silu=False):
    h = d["h"] if h is None else h
    w = d["conv_w"] if w is None else w
    bias = d["conv_bias"] if bias is None else bias
    tail = d.get("tail_in") if tail is None else tail
    y, so, _, _ = oracle.fused_forward(h, w, d["gamma"], d["theta"], eps, tau, bias=bias, clamp_silu=clamp_silu,
                                       tail_in=tail, state_in=d["state_in"])
    return float(np.sum((np.conj(d["G"].astype(np.complex128)) * y).real) +
                 np.sum((np.conj(d["dstate_out"]) * so).real))


def fd(f, arr, idx, step=2.0 ** -13):
    hi, lo = arr.copy(), arr.copy()
    hi[idx] += np.float32(step)
    lo[idx] -= np.float32(step)
    return (f(hi) - f(lo)) / (float(hi[idx]) - float(lo[idx]))


@pytest.mark.parametrize("clamp_silu", [False, True])
@pytest.mark.parametrize("Kc", [1, 3, 4])
def test_fused_backward_by_finite_differences_all_gates_open(Kc, clamp_silu):
    d = setup(Kc=Kc)
    g = oracle.fused_backward(d["h"], d["conv_w"], d["gamma"], d["theta"], d["G"], 0.0, -np.inf, bias=d["conv_bias"],
                              clamp_silu=clamp_silu, tail_in=d.get("tail_in"), state_in=d["state_in"],
                              dstate_out=d["dstate_out"])
    kw = dict(clamp_silu=clamp_silu)
    for idx in [(0, 0, 0), (1, 5, 2), (0, 23, 4), (1, 22, 1), (0, 11, 3)]:
        assert g["dh"][idx] == pytest.approx(fd(lambda a: loss(d, h=a, **kw), d["h"], idx), rel=2e-4, abs=2e-6)
    for c in range(5):
        for k in range(Kc):
            assert g["dw"][c, k] == pytest.approx(fd(lambda a: loss(d, w=a, **kw), d["conv_w"], (c, k)), rel=2e-4, abs=2e-5)
        assert g["dbias"][c] == pytest.approx(fd(lambda a: loss(d, bias=a, **kw), d["conv_bias"], (c,)), rel=2e-4, abs=2e-5)
    if Kc > 1:
        for idx in [(0, 0, 0), (1, Kc - 2, 3)]:
            assert g["dtail_in"][idx] == pytest.approx(fd(lambda a: loss(d, tail=a, **kw), d["tail_in"], idx), rel=2e-4, abs=2e-6)


def test_clamp_blocks_the_gradient_outside_its_interval():
    d = setup(L=6, C=3, Kc=1, with_tail=False)
    d["conv_w"][:] = 1.0
    d["conv_bias"][:] = 0.0
    d["h"][0, 2, 1] = 80.0                       # beyond the +-50 clamp: no gradient reaches this input
    dz = np.ones((2, 6, 3), np.complex128)
    g = oracle.prelude_bwd(d["h"], d["conv_w"], dz, bias=d["conv_bias"], clamp_silu=True)
    assert g["dh"][0, 2, 1] == 0.0 and np.count_nonzero(g["dh"]) == g["dh"].size - 1


def test_straight_through_gate_passes_magnitude_gradient_only():
    # Closed gate: the forward value is 0, the magnitude gradient flows as if the gate were open
    # and the phase gradient vanishes.  Stated without the oracle's formula: the closed-gate
    # gradient equals the open-gate gradient (pinned above by finite differences) of dz projected
    # on the push direction e^{i phase}, for which the phase term is zero by construction.
    d = setup(L=16, C=4)
    h, w, b = d["h"], d["conv_w"], d["conv_bias"]
    dz = d["G"].astype(np.complex128)
    z_open, _, _ = oracle.prelude(h, w, b, tail_in=d["tail_in"], gate_eps=0.0, gate_tau=-np.inf)
    dirn = z_open / np.abs(z_open)
    dz_proj = (np.conj(dz) * dirn).real * dirn
    closed = oracle.prelude_bwd(h, w, dz, bias=b, tail_in=d["tail_in"], gate_eps=0.5, gate_tau=np.inf)
    open_proj = oracle.prelude_bwd(h, w, dz_proj, bias=b, tail_in=d["tail_in"], gate_eps=0.0, gate_tau=-np.inf)
    for k in ("dh", "dw", "dbias", "dtail_in"):
        assert np.allclose(closed[k], open_proj[k], rtol=1e-10, atol=1e-12), k
    # and a mixed mask: each element follows its own gate
    tau = inputs.gate_tau(0.1)
    _, mask, _ = oracle.prelude(h, w, b, tail_in=d["tail_in"], gate_eps=0.1, gate_tau=tau)
    assert 0 < mask.sum() < mask.size
    mixed = oracle.prelude_bwd(h, w, dz, bias=b, tail_in=d["tail_in"], gate_eps=0.1, gate_tau=tau)
    dz_mix = np.where(mask.astype(bool), dz, dz_proj)
    ref = oracle.prelude_bwd(h, w, dz_mix, bias=b, tail_in=d["tail_in"], gate_eps=0.0, gate_tau=-np.inf)
    assert np.allclose(mixed["dh"], ref["dh"], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("split", [10, 1, 22])
def test_chunked_backward_equals_unchunked(split):
    d = setup(L=24, C=4, with_tail=False)
    tau = inputs.gate_tau(0.1)
    args = dict(gate_eps=0.1, gate_tau=tau, bias=d["conv_bias"])
    full = oracle.fused_backward(d["h"], d["conv_w"], d["gamma"], d["theta"], d["G"], state_in=d["state_in"],
                                 dstate_out=d["dstate_out"], **args)
    h1, h2 = d["h"][:, :split], d["h"][:, split:]
    # forward through the two chunks to get the state and history the second one starts from
    _, s1, _, tail1 = oracle.fused_forward(h1, d["conv_w"], d["gamma"], d["theta"], 0.1, tau, bias=d["conv_bias"],
                                           state_in=d["state_in"])
    b2 = oracle.fused_backward(h2, d["conv_w"], d["gamma"], d["theta"], d["G"][:, split:], tail_in=tail1, state_in=s1,
                               dstate_out=d["dstate_out"], **args)
    b1 = oracle.fused_backward(h1, d["conv_w"], d["gamma"], d["theta"], d["G"][:, :split], state_in=d["state_in"],
                               dstate_out=b2["dstate_in"], dtail_out=b2["dtail_in"], **args)
    assert np.allclose(np.concatenate([b1["dh"], b2["dh"]], axis=1), full["dh"], rtol=1e-9, atol=1e-11)
    assert np.allclose(b1["dw"] + b2["dw"], full["dw"], rtol=1e-9, atol=1e-11)
    assert np.allclose(b1["dbias"] + b2["dbias"], full["dbias"], rtol=1e-9, atol=1e-11)
    assert np.allclose(b1["dgamma"] + b2["dgamma"], full["dgamma"], rtol=1e-9, atol=1e-11)
    assert np.allclose(b1["dstate_in"], full["dstate_in"], rtol=1e-9, atol=1e-11)
