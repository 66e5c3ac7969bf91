"""Shared test helpers: the error metric and chunk utilities (no method arithmetic)."""
import numpy as np


def floored_rel_err(got, want, axes=None):
    """max |got - want| / max(|want|, rho) over complex moduli.

    Pure element-wise relative error is unattainable for sums with cancellation
    (the smallest of ~1e7 Rayleigh-distributed moduli is ~4e-4 of the RMS), so the
    denominator is floored at rho = RMS of |want| over ``axes`` (per channel for
    [B,L,C] outputs: axes=(0,1); all elements when ``axes`` is None).
    """
    got = np.asarray(got)
    want = np.asarray(want)
    if want.size == 0:
        return 0.0
    aw = np.abs(want).astype(np.float64)
    if axes is None:
        rho = np.sqrt(np.mean(aw ** 2))
    else:
        rho = np.sqrt(np.mean(aw ** 2, axis=axes, keepdims=True))
    den = np.maximum(aw, np.maximum(rho, 1e-300))
    return float(np.max(np.abs(got.astype(np.complex128) - want) / den))


def unpack_mask(words, C):
    """[.., ceil(C/32)] uint32 bit-packed (bit c%32 of word c//32) -> [.., C] uint8."""
    words = np.ascontiguousarray(words, dtype=np.uint32)
    bits = np.unpackbits(words.view(np.uint8).reshape(words.shape + (4,)),
                         axis=-1, bitorder="little")
    bits = bits.reshape(words.shape[:-1] + (words.shape[-1] * 32,))
    return bits[..., :C]
