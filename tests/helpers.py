"""Shared test helpers: the error metric and chunk utilities (no method arithmetic)."""
import os

import numpy as np


# Margins seen by every comparison of this session: (test id, floored maximum, unfloored median).
MARGINS = []


def floored_rel_err(got, want, axes="auto"):
    """max |got - want| / max(|want|, rho) over complex moduli.

    Pure element-wise relative error is unattainable for sums with cancellation
    (the smallest of ~1e7 Rayleigh-distributed moduli is ~4e-4 of the RMS), so the
    denominator is floored at rho = RMS of |want| over ``axes``.  The default floors per
    channel for arrays shaped [B, L, ...] (RMS over batch and time: axes (0, 1)) and over all
    elements for states and parameter gradients ([B, C], [C]); ``axes=None`` forces the latter.
    Every call also records the unfloored median of |got - want| / |want| next to the floored
    maximum, so that a test run shows how far below its tolerance each path sits.
    """
    got = np.asarray(got)
    want = np.asarray(want)
    if want.size == 0:
        return 0.0
    if isinstance(axes, str):
        axes = (0, 1) if want.ndim >= 3 else None
    aw = np.abs(want).astype(np.float64)
    if axes is None:
        rho = np.sqrt(np.mean(aw ** 2))
    else:
        rho = np.sqrt(np.mean(aw ** 2, axis=axes, keepdims=True))
    diff = np.abs(got.astype(np.complex128) - want)
    err = float(np.max(diff / np.maximum(aw, np.maximum(rho, 1e-300))))
    nz = aw > 0
    med = float(np.median(diff[nz] / aw[nz])) if nz.any() else 0.0
    test = os.environ.get("PYTEST_CURRENT_TEST", "").split(" ")[0]
    MARGINS.append((test, err, med))
    return err


def unpack_mask(words, C):
    """[.., ceil(C/32)] uint32 bit-packed (bit c%32 of word c//32) -> [.., C] uint8."""
    words = np.ascontiguousarray(words, dtype=np.uint32)
    bits = np.unpackbits(words.view(np.uint8).reshape(words.shape + (4,)),
                         axis=-1, bitorder="little")
    bits = bits.reshape(words.shape[:-1] + (words.shape[-1] * 32,))
    return bits[..., :C]
