"""Seeded synthetic inputs shaped like a CAWN Resonance Layer at d=768.

This module holds input generation only -- none of the method's arithmetic --
so that the CUDA path and the CPU oracle can be fed the same arrays without
sharing any code of their own.  Everything is drawn from one
``numpy.random.default_rng(seed)`` in a fixed order (magnitudes, phases,
retention, rotation, then extras), computed in float64 and rounded once to
float32.

The paper's own workloads are activations of a trained 150M-parameter model on
a web corpus; neither is available, so these arrays take the *shapes* and value
ranges of such a layer and stand in for it.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    B: int
    L: int
    H: int
    F: int
    gamma_lo: float
    gamma_hi: float
    gate_eps: float
    seed: int
    chunk: int = 0          # chunked prefill: tokens per call (0 = one call)
    conv_k: int = 0         # fused path: conv taps (0 = Cartesian pushes)

    @property
    def C(self) -> int:
        return self.H * self.F


# The five benchmark workloads.
CONFIGS = (
    Config("cfg0_tiny_fwd", B=1, L=256, H=4, F=16, gamma_lo=0.9, gamma_hi=0.999,
           gate_eps=0.1, seed=0),
    Config("cfg1_train_fwd", B=8, L=2048, H=12, F=64, gamma_lo=0.95, gamma_hi=0.9999,
           gate_eps=0.1, seed=1),
    Config("cfg2_chunked_prefill", B=1, L=2_000_000, H=12, F=64, gamma_lo=0.95,
           gamma_hi=0.9999, gate_eps=0.1, seed=2, chunk=4096),
    Config("cfg3_bwd", B=8, L=4096, H=12, F=64, gamma_lo=0.95, gamma_hi=0.9999,
           gate_eps=0.1, seed=3),
    Config("cfg4_fused", B=16, L=8192, H=12, F=64, gamma_lo=0.95, gamma_hi=0.9999,
           gate_eps=0.1, seed=4, conv_k=4),
)


def log_uniform(rng, lo, hi, n):
    """exp(U(ln lo, ln hi)) -- 'log-uniform in [lo, hi]' read literally."""
    return np.exp(rng.uniform(math.log(lo), math.log(hi), n))


def paper_theta(C):
    """The paper's fixed rotation angles theta_j = 10000^(-2j/C), j = 0..C-1."""
    j = np.arange(C, dtype=np.float64)
    return (10000.0 ** (-2.0 * j / C)).astype(np.float32)


def polar_pushes(rng, shape):
    """Complex64 pushes with magnitude U[0,1) and phase U[-pi,pi)."""
    m = rng.uniform(0.0, 1.0, shape)
    ph = rng.uniform(-math.pi, math.pi, shape)
    out = np.empty(shape, np.complex64)
    out.real = (m * np.cos(ph)).astype(np.float32)
    out.imag = (m * np.sin(ph)).astype(np.float32)
    return out


def scan_inputs(B, L, C, seed, gamma_lo=0.95, gamma_hi=0.9999,
                theta_lo=0.0, theta_hi=0.1, with_state=False, with_grad=False):
    """Inputs of the Cartesian forward (and backward) scan.

    Draw order: magnitudes, phases (inside polar_pushes), gamma, theta, then the
    optional extras state_in, grad_y, grad_state_out.
    """
    rng = np.random.default_rng(seed)
    d = {"p": polar_pushes(rng, (B, L, C))}
    d["gamma"] = log_uniform(rng, gamma_lo, gamma_hi, C).astype(np.float32)
    d["theta"] = rng.uniform(theta_lo, theta_hi, C).astype(np.float32)
    if with_state:
        s = rng.normal(0.0, 2.0, (B, C, 2))
        d["state_in"] = (s[..., 0] + 1j * s[..., 1]).astype(np.complex64)
    if with_grad:
        g = rng.normal(0.0, 1.0, (B, L, C, 2)).astype(np.float32)
        d["grad_y"] = g.view(np.complex64).reshape(B, L, C)
        gs = rng.normal(0.0, 1.0, (B, C, 2)).astype(np.float32)
        d["grad_state_out"] = gs.view(np.complex64).reshape(B, C)
    return d


def config_inputs(cfg: Config, with_state=False):
    """Inputs for one of CONFIGS (cfg 2: use :func:`prefill_stream` instead)."""
    if cfg.conv_k:
        return fused_inputs(cfg.B, cfg.L, cfg.C, cfg.seed, cfg.conv_k,
                            cfg.gamma_lo, cfg.gamma_hi)
    return scan_inputs(cfg.B, cfg.L, cfg.C, cfg.seed, cfg.gamma_lo, cfg.gamma_hi,
                       with_state=with_state, with_grad=(cfg.name == "cfg3_bwd"))


def fused_inputs(B, L, C, seed, conv_k=4, gamma_lo=0.95, gamma_hi=0.9999,
                 with_tail=False, with_bias=False):
    """Inputs of the fused mixing path: hidden states N(0,1), conv weights N(0, std 0.5)."""
    rng = np.random.default_rng(seed)
    d = {"h": rng.normal(0.0, 1.0, (B, L, C)).astype(np.float32)}
    d["gamma"] = log_uniform(rng, gamma_lo, gamma_hi, C).astype(np.float32)
    d["theta"] = rng.uniform(0.0, 0.1, C).astype(np.float32)
    d["conv_w"] = rng.normal(0.0, 0.5, (C, conv_k)).astype(np.float32)
    if with_tail:
        d["tail_in"] = rng.normal(0.0, 1.0, (B, conv_k - 1, C)).astype(np.float32)
    if with_bias:
        d["conv_bias"] = rng.normal(0.0, 0.5, C).astype(np.float32)
    return d


def dynamic_retention_inputs(B, L, H, F, seed):
    """Per-head retention logits and the static per-harmonic bias (+3 -> 0 over F)."""
    rng = np.random.default_rng(seed)
    logit = rng.normal(2.0, 1.5, (B, L, H)).astype(np.float32)
    bias = np.linspace(3.0, 0.0, F).astype(np.float32)
    return {"gamma_logit": logit, "freq_bias": bias}


def prefill_stream(cfg: Config, total=None, chunk=None):
    """Yield (gamma, theta) once, then complex64 chunks [B, n, C] of a long stream.

    The stream is drawn chunk by chunk from one generator, so any consumer that
    uses the same chunk size sees the same tokens.
    """
    total = cfg.L if total is None else total
    chunk = (cfg.chunk or total) if chunk is None else chunk
    rng = np.random.default_rng(cfg.seed)
    gamma = log_uniform(rng, cfg.gamma_lo, cfg.gamma_hi, cfg.C).astype(np.float32)
    theta = rng.uniform(0.0, 0.1, cfg.C).astype(np.float32)
    yield gamma, theta
    done = 0
    while done < total:
        n = min(chunk, total - done)
        yield polar_pushes(rng, (cfg.B, n, cfg.C))
        done += n


def gate_tau(gate_eps: float) -> np.float32:
    """logit(eps) rounded once to fp32: the fused path's gate threshold on the conv output."""
    if gate_eps <= 0.0:
        return np.float32(-np.inf)
    if gate_eps >= 1.0:
        return np.float32(np.inf)
    return np.float32(math.log(gate_eps / (1.0 - gate_eps)))


def to_bf16(a):
    """Round a float array to bfloat16 (nearest even).  Returns (bits uint16, the same values widened
    back to float32); complex input is treated as (re, im) pairs.  Storage conversion only: the
    bf16-input parity cases feed the bits to the device and the widened values to the oracle."""
    a = np.ascontiguousarray(a)
    cplx = np.iscomplexobj(a)
    f = a.astype(np.complex64).view(np.float32) if cplx else a.astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    wide = (r.astype(np.uint32) << 16).view(np.float32)
    if cplx:
        return r.reshape(a.shape + (2,)), wide.view(np.complex64).reshape(a.shape)
    return r.reshape(a.shape), wide.reshape(a.shape)


def from_bf16(bits):
    """bfloat16 bits (uint16) -> float32; a trailing axis of 2 is NOT folded into complex here."""
    return (np.ascontiguousarray(bits).astype(np.uint32) << 16).view(np.float32)
