"""The input module's bfloat16 storage conversion against torch's (no GPU)."""
import numpy as np

from paper_2604_04250_b200 import inputs


def test_to_bf16_is_round_to_nearest_even():
    import torch
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=4000), rng.normal(size=100) * 1e-20, [0.0, -0.0, 1.0, 1.00390625, 1.01171875]]).astype(np.float32)
    bits, wide = inputs.to_bf16(x)
    t = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(t.view(torch.int16).numpy().view(np.uint16), bits)
    assert np.array_equal(t.float().numpy(), wide)
    assert np.array_equal(inputs.from_bf16(bits), wide)
    z = (x[:2000] + 1j * x[2000:4000]).astype(np.complex64)
    zb, zw = inputs.to_bf16(z)
    assert zb.shape == (2000, 2) and np.array_equal(zw.real, wide[:2000]) and np.array_equal(zw.imag, wide[2000:4000])
