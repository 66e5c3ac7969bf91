"""CPU fp64 oracle for CAWN phase accumulation -- TEST INFRASTRUCTURE ONLY.

Thin ctypes marshalling around ``cawn_oracle.c`` (plain sequential C, double
precision).  Only the tests, the smoke check and the benchmark's CPU-baseline
leg may import this package; the CUDA library and its binding never do, and
this package imports nothing of theirs.

Functions mirror the steps of the path:

* :func:`gate`        hard-threshold gate on Cartesian pushes
* :func:`prelude`     causal depthwise conv -> phasor map -> gate -> push
* :func:`scan`        the recurrence of Eq. (phase_accum_r/i), clamp, state
* :func:`scan_bwd`    reverse-time adjoint with parameter gradients
* :func:`prelude_bwd` backward of the prelude (conv, phasor map, straight-through gate)
* :func:`wave_synthesis`, :func:`ear_conv`  planar Z of Eq. (wave_synth) and the depthwise
  convolution across the harmonics that opens the SwiGLU Ear
* :func:`forward`, :func:`fused_forward`, :func:`fused_backward`  compositions of the above

No function here is "parity unpinned": see ``tests/test_oracle_*.py``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cawn_oracle.c")
_LIB = os.path.join(_HERE, "libcawn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with the host C compiler (no CUDA involved)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(
        ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fvisibility=hidden",
         "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _ptr(a, dtype):
    if a is None:
        return None
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _as_pairs(a, dtype):
    """complex array [...]  ->  real array [..., 2] of ``dtype`` (a view when possible)."""
    if a is None:
        return None
    a = np.asarray(a)
    if np.iscomplexobj(a):
        want = np.complex64 if dtype == np.float32 else np.complex128
        a = np.ascontiguousarray(a, dtype=want)
        return a.view(dtype).reshape(a.shape + (2,))
    return np.ascontiguousarray(a, dtype=dtype)


def _as_complex(a):
    return a.view(np.complex128).reshape(a.shape[:-1])


def gate(p, gate_eps):
    """Hard gate on complex64 pushes ``p`` (any shape).  Returns (z complex128, mask uint8)."""
    pp = _as_pairs(p, np.float32)
    n = pp.size // 2
    z = np.empty(pp.shape, np.float64)
    mask = np.empty(pp.shape[:-1], np.uint8)
    _load().cawn_oracle_gate(
        ctypes.c_int64(n), _ptr(pp, np.float32), ctypes.c_float(gate_eps),
        _ptr(z, np.float64), _ptr(mask, np.uint8))
    return _as_complex(z), mask


def scan(z, theta, gamma=None, gamma_logit=None, freq_bias=None, H=None,
         state_in=None, clamp_abs=0.0, want_P=False):
    """Sequential recurrence over gated pushes ``z`` [B,L,C] complex128.

    Static retention: ``gamma`` [C].  Dynamic: ``gamma_logit`` [B,L,H] and
    ``freq_bias`` [F] with C = H*F.  Returns (y, state_out[, P]) as complex128;
    ``y`` is clamped when ``clamp_abs`` > 0, ``state_out`` and ``P`` never are.
    """
    zz = _as_pairs(z, np.float64)
    B, L, C = zz.shape[:3]
    if gamma is not None:
        Hh, F = (H, C // H) if H else (1, C)
    else:
        Hh = gamma_logit.shape[-1]
        F = C // Hh
    assert Hh * F == C
    y = np.empty(zz.shape, np.float64)
    so = np.empty((B, C, 2), np.float64)
    P = np.empty(zz.shape, np.float64) if want_P else None
    si = _as_pairs(state_in, np.float64)
    g, th = _f32(gamma), _f32(theta)
    gl, fb = _f32(gamma_logit), _f32(freq_bias)
    _load().cawn_oracle_scan(
        ctypes.c_int(B), ctypes.c_int64(L), ctypes.c_int(Hh), ctypes.c_int(F),
        _ptr(zz, np.float64), _ptr(g, np.float32), _ptr(th, np.float32),
        _ptr(gl, np.float32), _ptr(fb, np.float32),
        _ptr(si, np.float64), ctypes.c_double(clamp_abs),
        _ptr(P, np.float64), _ptr(y, np.float64), _ptr(so, np.float64))
    out = (_as_complex(y), _as_complex(so))
    return out + ((_as_complex(P),) if want_P else ())


def prelude(h, w, bias=None, clamp_silu=False, tail_in=None,
            gate_eps=0.0, gate_tau=-np.inf):
    """Conv prelude + phasor map + gate + push.  ``h`` [B,L,C] fp32, ``w`` [C,Kc].

    Returns (z complex128 [B,L,C], mask uint8 [B,L,C], tail_out fp32 [B,Kc-1,C]).
    """
    hh, ww, bb, ti = _f32(h), _f32(w), _f32(bias), _f32(tail_in)
    B, L, C = hh.shape
    Kc = ww.shape[1]
    assert ww.shape[0] == C
    z = np.empty((B, L, C, 2), np.float64)
    mask = np.empty((B, L, C), np.uint8)
    to = np.empty((B, Kc - 1, C), np.float32)
    _load().cawn_oracle_prelude(
        ctypes.c_int(B), ctypes.c_int64(L), ctypes.c_int(C),
        _ptr(hh, np.float32), _ptr(ww, np.float32), _ptr(bb, np.float32),
        ctypes.c_int(Kc), ctypes.c_int(int(bool(clamp_silu))),
        _ptr(ti, np.float32), ctypes.c_float(gate_eps), ctypes.c_float(gate_tau),
        _ptr(z, np.float64), _ptr(mask, np.uint8), _ptr(to, np.float32))
    return _as_complex(z), mask, to


def scan_bwd(z, theta, G, gamma=None, gamma_logit=None, freq_bias=None, H=None,
             state_in=None, dstate_out=None, grad_clamp_abs=0.0):
    """Reverse-time adjoint.  Returns a dict with dp, dstate_in (complex128),
    dtheta and either dgamma (static) or dgamma_logit, dfreq_bias (dynamic)."""
    zz = _as_pairs(z, np.float64)
    B, L, C = zz.shape[:3]
    static = gamma is not None
    if static:
        Hh, F = (H, C // H) if H else (1, C)
    else:
        Hh = gamma_logit.shape[-1]
        F = C // Hh
    GG = _as_pairs(G, np.float32)
    dp = np.empty(zz.shape, np.float64)
    dth = np.empty(C, np.float64)
    dsi = np.empty((B, C, 2), np.float64)
    dg = np.empty(C, np.float64) if static else None
    dgl = None if static else np.empty((B, L, Hh), np.float64)
    dfb = None if static else np.empty(F, np.float64)
    si, dso = _as_pairs(state_in, np.float64), _as_pairs(dstate_out, np.float64)
    g, th = _f32(gamma), _f32(theta)
    gl, fb = _f32(gamma_logit), _f32(freq_bias)
    _load().cawn_oracle_scan_bwd(
        ctypes.c_int(B), ctypes.c_int64(L), ctypes.c_int(Hh), ctypes.c_int(F),
        _ptr(zz, np.float64), _ptr(g, np.float32), _ptr(th, np.float32),
        _ptr(gl, np.float32), _ptr(fb, np.float32), _ptr(si, np.float64),
        _ptr(GG, np.float32), _ptr(dso, np.float64), ctypes.c_double(grad_clamp_abs),
        _ptr(dp, np.float64), _ptr(dg, np.float64), _ptr(dth, np.float64),
        _ptr(dsi, np.float64), _ptr(dgl, np.float64), _ptr(dfb, np.float64))
    out = {"dp": _as_complex(dp), "dtheta": dth, "dstate_in": _as_complex(dsi)}
    if static:
        out["dgamma"] = dg
    else:
        out["dgamma_logit"] = dgl
        out["dfreq_bias"] = dfb
    return out


def wave_synthesis(y, H, K):
    """Eq. (wave_synth): Z_t = Concat(P^(r)_t, P^(i)_t).  ``y`` [B,L,H*K] complex ->
    Z [B,L,2,H,K] float64: all real parts (head-major), then all imaginary parts."""
    y = np.asarray(y, dtype=np.complex128)
    B, L, C = y.shape
    assert C == H * K
    Z = np.empty((B, L, 2, H, K), dtype=np.float64)
    Z[:, :, 0] = y.real.reshape(B, L, H, K)
    Z[:, :, 1] = y.imag.reshape(B, L, H, K)
    return Z


def ear_conv(y, ear_w, ear_bias, H, K):
    """Front of the Convolutional SwiGLU Ear (Section "Projection to Hidden State"): Z is viewed
    as 2H feature channels (real heads, then imaginary heads) over K positions (the harmonics),
    and each channel is convolved along K with its own taps.

    ``ear_w`` [2H, Ke] with Ke odd, ``ear_bias`` [2H] or None.  The paper gives neither Ke nor
    the padding; taken here: zero padding of (Ke-1)/2 on both sides (output length K) and the
    cross-correlation convention of a Conv1d layer,
        out[q, k] = bias[q] + sum_j w[q, j] Z[q, k + j - (Ke-1)/2].
    Returns Z_conv [B,L,2,H,K] float64 (flattening its last three axes gives the 2HK-wide row).
    """
    Z = wave_synthesis(y, H, K)
    w = np.asarray(ear_w, dtype=np.float64)
    Q, Ke = w.shape
    assert Q == 2 * H and Ke % 2 == 1
    r = (Ke - 1) // 2
    B, L = Z.shape[:2]
    Zq = Z.reshape(B, L, Q, K)
    pad = np.zeros((B, L, Q, K + 2 * r), dtype=np.float64)
    pad[..., r:r + K] = Zq
    out = np.zeros((B, L, Q, K), dtype=np.float64)
    if ear_bias is not None:
        out += np.asarray(ear_bias, dtype=np.float64)[None, None, :, None]
    for j in range(Ke):
        out += w[None, None, :, j, None] * pad[..., j:j + K]
    return out.reshape(B, L, 2, H, K)


def forward(p, gamma, theta, gate_eps, state_in=None, clamp_abs=0.0, **kw):
    """gate -> scan on complex64 pushes.  Returns (y, state_out, mask)."""
    z, mask = gate(p, gate_eps)
    y, so = scan(z, theta, gamma=gamma, state_in=state_in, clamp_abs=clamp_abs, **kw)
    return y, so, mask


def fused_forward(h, w, gamma, theta, gate_eps, gate_tau, bias=None,
                  clamp_silu=False, tail_in=None, state_in=None, clamp_abs=0.0, **kw):
    """prelude -> scan on fp32 hidden states.  Returns (y, state_out, mask, tail_out).
    ``gamma=None`` with ``gamma_logit=, freq_bias=, H=`` gives the time-varying retention."""
    z, mask, tail = prelude(h, w, bias, clamp_silu, tail_in, gate_eps, gate_tau)
    y, so = scan(z, theta, gamma=gamma, state_in=state_in, clamp_abs=clamp_abs, **kw)
    return y, so, mask, tail


def prelude_bwd(h, w, dz, bias=None, clamp_silu=False, tail_in=None, gate_eps=0.0, gate_tau=-np.inf,
                dtail_out=None):
    """Backward of :func:`prelude` for a push gradient ``dz`` [B,L,C] complex.

    Returns a dict with dh [B,L,C], dw [C,Kc], dbias [C], dtail_in [B,Kc-1,C] (float64)."""
    hh, ww, bb, ti = _f32(h), _f32(w), _f32(bias), _f32(tail_in)
    B, L, C = hh.shape
    Kc = ww.shape[1]
    dzz = _as_pairs(np.asarray(dz, dtype=np.complex128), np.float64)
    dto = _f64(dtail_out)
    dh = np.empty((B, L, C), np.float64)
    dw = np.empty((C, Kc), np.float64)
    db = np.empty(C, np.float64)
    dti = np.empty((B, Kc - 1, C), np.float64)
    _load().cawn_oracle_prelude_bwd(
        ctypes.c_int(B), ctypes.c_int64(L), ctypes.c_int(C),
        _ptr(hh, np.float32), _ptr(ww, np.float32), _ptr(bb, np.float32),
        ctypes.c_int(Kc), ctypes.c_int(int(bool(clamp_silu))),
        _ptr(ti, np.float32), ctypes.c_float(gate_eps), ctypes.c_float(gate_tau),
        _ptr(dzz, np.float64), _ptr(dto, np.float64),
        _ptr(dh, np.float64), _ptr(dw, np.float64), _ptr(db, np.float64), _ptr(dti, np.float64))
    return {"dh": dh, "dw": dw, "dbias": db, "dtail_in": dti}


def fused_backward(h, w, gamma, theta, G, gate_eps, gate_tau, bias=None, clamp_silu=False, tail_in=None,
                   state_in=None, dstate_out=None, dtail_out=None, **kw):
    """prelude -> scan forward, then scan_bwd -> prelude_bwd.  Returns the union of both dicts.
    ``gamma=None`` with ``gamma_logit=, freq_bias=, H=`` gives the time-varying retention."""
    z, mask, _ = prelude(h, w, bias, clamp_silu, tail_in, gate_eps, gate_tau)
    out = scan_bwd(z, theta, G, gamma=gamma, state_in=state_in, dstate_out=dstate_out, **kw)
    out.update(prelude_bwd(h, w, out["dp"], bias, clamp_silu, tail_in, gate_eps, gate_tau, dtail_out))
    return out
