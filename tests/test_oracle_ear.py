"""Pins for the oracle's wave synthesis and Ear convolution (no GPU): the layout of
Eq. (wave_synth), a Conv1d library routine (the layer the paper names), numpy.correlate per
channel, and structural properties (heads do not mix, zero padding at both ends)."""
import numpy as np

import oracle


def _y(B, L, H, K, seed):
    rng = np.random.default_rng(seed)
    return (rng.normal(size=(B, L, H * K)) + 1j * rng.normal(size=(B, L, H * K))).astype(np.complex64)


def test_wave_synthesis_is_concat_of_real_and_imaginary():
    H, K = 3, 8
    y = _y(2, 5, H, K, 1)
    Z = oracle.wave_synthesis(y, H, K).reshape(2, 5, 2 * H * K)
    assert np.array_equal(Z[..., :H * K], y.real.astype(np.float64))
    assert np.array_equal(Z[..., H * K:], y.imag.astype(np.float64))


def test_identity_taps_return_planar_z():
    H, K = 2, 16
    y = _y(1, 7, H, K, 2)
    w = np.zeros((2 * H, 3)); w[:, 1] = 1.0
    assert np.array_equal(oracle.ear_conv(y, w, None, H, K), oracle.wave_synthesis(y, H, K))


def test_matches_depthwise_conv1d_layer():
    import torch
    for (H, K, Ke, seed) in [(3, 16, 3, 3), (2, 64, 3, 4), (4, 5, 5, 5), (1, 1, 3, 6), (2, 7, 1, 7)]:
        y = _y(2, 4, H, K, seed)
        rng = np.random.default_rng(seed + 100)
        w, bias = rng.normal(size=(2 * H, Ke)), rng.normal(size=2 * H)
        got = oracle.ear_conv(y, w, bias, H, K)
        Z = torch.from_numpy(np.concatenate([y.real, y.imag], axis=-1).astype(np.float64))     # [B,L,2HK]
        x = Z.reshape(-1, 2 * H, K)                                                           # harmonics as length
        ref = torch.nn.functional.conv1d(x, torch.from_numpy(w)[:, None, :], torch.from_numpy(bias),
                                         padding=(Ke - 1) // 2, groups=2 * H)
        assert np.allclose(got.reshape(-1, 2 * H, K), ref.numpy(), rtol=1e-13, atol=1e-13)


def test_matches_numpy_correlate_per_channel():
    H, K = 2, 12
    y = _y(1, 2, H, K, 8)
    rng = np.random.default_rng(9)
    w = rng.normal(size=(2 * H, 3))
    got = oracle.ear_conv(y, w, None, H, K).reshape(2, 2 * H, K)
    Z = oracle.wave_synthesis(y, H, K).reshape(2, 2 * H, K)
    for t in range(2):
        for q in range(2 * H):
            assert np.allclose(got[t, q], np.correlate(Z[t, q], w[q], mode="same"), rtol=1e-13, atol=1e-13)


def test_heads_and_parts_do_not_mix_and_edges_are_zero_padded():
    H, K = 3, 8
    y = np.zeros((1, 1, H * K), dtype=np.complex64)
    y[0, 0, 1 * K + 0] = 2.0            # head 1, harmonic 0, real part only
    y[0, 0, 1 * K + K - 1] += 3.0j      # head 1, last harmonic, imaginary part only
    w = np.tile(np.array([10.0, 1.0, 100.0]), (2 * H, 1))
    out = oracle.ear_conv(y, w, None, H, K)[0, 0]
    exp = np.zeros((2, H, K))
    exp[0, 1, 0], exp[0, 1, 1] = 2.0, 20.0          # centre tap at k=0, left tap seen from k=1; nothing leaks into head 0
    exp[1, 1, K - 1], exp[1, 1, K - 2] = 3.0, 300.0 # centre tap at k=K-1, right tap seen from k=K-2; nothing leaks into head 2
    assert np.array_equal(out, exp)
