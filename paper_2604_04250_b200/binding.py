"""ctypes binding of ``libcawn.so`` -- argument marshalling only.

Function names and argument order follow ``include/cawn.h``.  Tensors are torch CUDA tensors
(used purely as device memory) or ``None``; complex64 tensors are passed as they are
(interleaved re, im).  Every step of the path runs in the library's CUDA kernels: there is no
CPU or eager fallback, and a missing library is an error.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcawn.so")

CAWN_OK = 0
CAWN_ERR_INVALID_ARG = -1
CAWN_ERR_NULL_POINTER = -2
CAWN_ERR_MISALIGNED = -3
CAWN_ERR_UNSUPPORTED = -4
CAWN_ERR_WORKSPACE_TOO_SMALL = -5
CAWN_ERR_CUDA = -6
CAWN_ERR_STATIC_TOO_LARGE = -7
CAWN_STATIC_SCRATCH_BYTES = 4 << 20
CAWN_ERR_CARRY_TIMEOUT = 1
CAWN_STATUS_NONFINITE = 2

CAWN_FLAG_PRELUDE_CLAMP_SILU = 1
CAWN_FLAG_RETENTION_DYNAMIC = 2
CAWN_FLAG_INPUT_INDEPENDENT = 4
CAWN_FLAG_INPUT_BF16 = 8
CAWN_FLAG_OUTPUT_BF16 = 16

CAWN_OP_FWD, CAWN_OP_BWD_SAVED, CAWN_OP_BWD_PUSHES, CAWN_OP_STATE, CAWN_OP_FWD_HOST, CAWN_OP_MIXING_BWD = range(6)
CAWN_SAVED_STATES, CAWN_SAVED_PUSHES = 0, 1

EXPORTS = (
    "cawn_status_string", "cawn_workspace_bytes", "cawn_workspace_init",
    "cawn_phase_accumulate_fwd", "cawn_phase_accumulate_bwd", "cawn_state_carry",
    "cawn_poll_status", "cawn_phase_accumulate_fwd_host", "cawn_phase_accumulate_fwd_static",
    "cawn_phase_accumulate_bwd_dynamic", "cawn_mixing_bwd", "cawn_phase_accumulate_fwd_ear",
    "cawn_workspace_set_wait_hook", "cawn_mixing_bwd_dynamic",
)


class cawn_params(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("B", ctypes.c_int32),
        ("L", ctypes.c_int64),
        ("H", ctypes.c_int32),
        ("F", ctypes.c_int32),
        ("gate_eps", ctypes.c_float),
        ("gate_tau", ctypes.c_float),
        ("clamp_abs", ctypes.c_float),
        ("grad_clamp_abs", ctypes.c_float),
        ("conv_k", ctypes.c_int32),
        ("flags", ctypes.c_uint32),
    ]


class CawnError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, status_string(status), status))


_lib = None


def lib():
    """Load ``libcawn.so`` (built in-tree by ``paper_2604_04250_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libcawn.so is missing: run `python -m paper_2604_04250_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, fp, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t
        pp = ctypes.POINTER(cawn_params)
        L.cawn_status_string.restype = ctypes.c_char_p
        L.cawn_status_string.argtypes = [ctypes.c_int]
        L.cawn_workspace_bytes.argtypes = [pp, ctypes.c_int, ctypes.POINTER(sz)]
        L.cawn_workspace_init.argtypes = [vp, sz, vp]
        L.cawn_phase_accumulate_fwd.argtypes = [pp, vp, fp, fp, fp, fp, fp, fp, vp, vp, vp, vp, vp, sz, vp]
        L.cawn_phase_accumulate_bwd.argtypes = [pp, vp, ctypes.c_int, fp, fp, vp, vp, vp, vp, fp, fp, vp, vp, sz, vp]
        L.cawn_phase_accumulate_bwd_dynamic.argtypes = [pp, vp, ctypes.c_int, fp, fp, fp, vp, vp, vp, vp, fp, fp, fp, vp, vp, sz, vp]
        L.cawn_mixing_bwd.argtypes = [pp, fp, fp, fp, fp, fp, vp, vp, vp, vp, fp, fp, fp, fp, fp, vp, vp, sz, vp]
        L.cawn_phase_accumulate_fwd_ear.argtypes = [pp, vp, fp, fp, fp, fp, fp, fp, vp, fp, fp, ctypes.c_int, fp, vp, vp, vp, sz, vp]
        L.cawn_mixing_bwd_dynamic.argtypes = [pp, fp, fp, fp, fp, fp, fp, vp, vp, vp, vp, fp, fp, fp, fp, fp, fp, vp, vp, sz, vp]
        L.cawn_state_carry.argtypes = [pp, vp, vp, ctypes.c_int64, fp, fp, vp, vp]
        L.cawn_poll_status.argtypes = [vp, vp]
        L.cawn_workspace_set_wait_hook.argtypes = [vp, ctypes.c_int, ctypes.c_uint, vp]
        L.cawn_phase_accumulate_fwd_host.argtypes = [pp, vp, fp, fp, vp, vp, vp, vp, vp, sz, vp]
        L.cawn_phase_accumulate_fwd_static.argtypes = [pp, vp, fp, fp, vp, vp, vp, vp, vp, vp]
        for name in EXPORTS:
            if name != "cawn_status_string":
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def make_params(B, L, H, F, gate_eps=0.0, gate_tau=0.0, clamp_abs=0.0, grad_clamp_abs=0.0,
                conv_k=0, flags=0):
    return cawn_params(ctypes.sizeof(cawn_params), B, L, H, F, gate_eps, gate_tau, clamp_abs,
                       grad_clamp_abs, conv_k, flags)


def status_string(status):
    return lib().cawn_status_string(int(status)).decode()


def _dp(t):
    """Device (or host) pointer of a tensor / numpy array / None."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def _check(rc, where):
    if rc != CAWN_OK:
        raise CawnError(rc, where)


def cawn_workspace_bytes(params, op):
    n = ctypes.c_size_t(0)
    _check(lib().cawn_workspace_bytes(ctypes.byref(params), op, ctypes.byref(n)), "cawn_workspace_bytes")
    return n.value


def cawn_workspace_init(workspace, stream=None):
    _check(lib().cawn_workspace_init(_dp(workspace), workspace.numel() * workspace.element_size(),
                                     _stream(stream)), "cawn_workspace_init")


def new_workspace(params, op, device="cuda"):
    """Allocate (with torch, as plain device memory) and initialise a workspace for `op`."""
    import torch
    n = cawn_workspace_bytes(params, op)
    ws = torch.empty(max(n, 256), dtype=torch.uint8, device=device)
    cawn_workspace_init(ws)
    return ws


def cawn_phase_accumulate_fwd(params, input, gamma, theta, y, workspace, conv_w=None, conv_bias=None,
                              gamma_logit=None, freq_bias=None, state_in=None, state_out=None,
                              gate_mask=None, stream=None):
    _check(lib().cawn_phase_accumulate_fwd(
        ctypes.byref(params), _dp(input), _dp(gamma), _dp(theta), _dp(conv_w), _dp(conv_bias),
        _dp(gamma_logit), _dp(freq_bias), _dp(state_in), _dp(y), _dp(state_out), _dp(gate_mask),
        _dp(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
        "cawn_phase_accumulate_fwd")


def cawn_phase_accumulate_fwd_ear(params, input, gamma, theta, ear_w, ear_k, z_conv, workspace, ear_bias=None,
                                  conv_w=None, conv_bias=None, gamma_logit=None, freq_bias=None, state_in=None,
                                  state_out=None, gate_mask=None, stream=None):
    _check(lib().cawn_phase_accumulate_fwd_ear(
        ctypes.byref(params), _dp(input), _dp(gamma), _dp(theta), _dp(conv_w), _dp(conv_bias), _dp(gamma_logit),
        _dp(freq_bias), _dp(state_in),
        _dp(ear_w), _dp(ear_bias), int(ear_k), _dp(z_conv), _dp(state_out), _dp(gate_mask),
        _dp(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
        "cawn_phase_accumulate_fwd_ear")


def cawn_phase_accumulate_bwd(params, saved, saved_kind, gamma, theta, grad_y, grad_p, workspace,
                              state_in=None, grad_state_out=None, grad_gamma=None, grad_theta=None,
                              grad_state_in=None, stream=None):
    _check(lib().cawn_phase_accumulate_bwd(
        ctypes.byref(params), _dp(saved), saved_kind, _dp(gamma), _dp(theta), _dp(state_in),
        _dp(grad_y), _dp(grad_state_out), _dp(grad_p), _dp(grad_gamma), _dp(grad_theta),
        _dp(grad_state_in), _dp(workspace), workspace.numel() * workspace.element_size(),
        _stream(stream)), "cawn_phase_accumulate_bwd")


def cawn_mixing_bwd_dynamic(params, h, conv_w, gamma_logit, freq_bias, theta, grad_y, grad_h, workspace, conv_bias=None,
                            saved_states=None, state_in=None, grad_state_out=None, grad_conv_w=None, grad_conv_bias=None,
                            grad_gamma_logit=None, grad_freq_bias=None, grad_theta=None, grad_state_in=None, stream=None):
    _check(lib().cawn_mixing_bwd_dynamic(
        ctypes.byref(params), _dp(h), _dp(conv_w), _dp(conv_bias), _dp(gamma_logit), _dp(freq_bias), _dp(theta),
        _dp(saved_states), _dp(state_in), _dp(grad_y), _dp(grad_state_out), _dp(grad_h), _dp(grad_conv_w),
        _dp(grad_conv_bias), _dp(grad_gamma_logit), _dp(grad_freq_bias), _dp(grad_theta), _dp(grad_state_in),
        _dp(workspace), workspace.numel() * workspace.element_size(), _stream(stream)), "cawn_mixing_bwd_dynamic")


def cawn_state_carry(params, state_prev, state_local, n_steps, gamma, theta, state_out, stream=None):
    _check(lib().cawn_state_carry(ctypes.byref(params), _dp(state_prev), _dp(state_local),
                                  int(n_steps), _dp(gamma), _dp(theta), _dp(state_out),
                                  _stream(stream)), "cawn_state_carry")


def cawn_workspace_set_wait_hook(workspace, withhold_tile, poll_bound, stream=None):
    _check(lib().cawn_workspace_set_wait_hook(_dp(workspace), int(withhold_tile), int(poll_bound), _stream(stream)),
           "cawn_workspace_set_wait_hook")


def cawn_poll_status(workspace, stream=None):
    return lib().cawn_poll_status(_dp(workspace), _stream(stream))


def cawn_phase_accumulate_fwd_host(params, p_host, gamma_host, theta_host, y_host, device_scratch,
                                   state_in_host=None, state_out_host=None, gate_mask_host=None,
                                   stream=None):
    _check(lib().cawn_phase_accumulate_fwd_host(
        ctypes.byref(params), _dp(p_host), _dp(gamma_host), _dp(theta_host), _dp(state_in_host),
        _dp(y_host), _dp(state_out_host), _dp(gate_mask_host), _dp(device_scratch),
        device_scratch.numel() * device_scratch.element_size(), _stream(stream)),
        "cawn_phase_accumulate_fwd_host")


def cawn_phase_accumulate_fwd_static(params, input, gamma, theta, y, state_in=None, state_out=None,
                                     gate_mask=None, device_status=None, stream=None):
    """Forward scan on the library's built-in scratch array: for callers that hold input and
    output buffers but cannot allocate a workspace.  One call at a time per device."""
    _check(lib().cawn_phase_accumulate_fwd_static(
        ctypes.byref(params), _dp(input), _dp(gamma), _dp(theta), _dp(state_in), _dp(y),
        _dp(state_out), _dp(gate_mask), _dp(device_status), _stream(stream)),
        "cawn_phase_accumulate_fwd_static")


def cawn_phase_accumulate_bwd_dynamic(params, saved, saved_kind, gamma_logit, freq_bias, theta, grad_y, grad_p,
                                      workspace, state_in=None, grad_state_out=None, grad_gamma_logit=None,
                                      grad_freq_bias=None, grad_theta=None, grad_state_in=None, stream=None):
    _check(lib().cawn_phase_accumulate_bwd_dynamic(
        ctypes.byref(params), _dp(saved), saved_kind, _dp(gamma_logit), _dp(freq_bias), _dp(theta),
        _dp(state_in), _dp(grad_y), _dp(grad_state_out), _dp(grad_p), _dp(grad_gamma_logit),
        _dp(grad_freq_bias), _dp(grad_theta), _dp(grad_state_in), _dp(workspace),
        workspace.numel() * workspace.element_size(), _stream(stream)), "cawn_phase_accumulate_bwd_dynamic")


def cawn_mixing_bwd(params, h, conv_w, gamma, theta, grad_y, grad_h, workspace, conv_bias=None, saved_states=None,
                    state_in=None, grad_state_out=None, grad_conv_w=None, grad_conv_bias=None, grad_gamma=None,
                    grad_theta=None, grad_state_in=None, stream=None):
    _check(lib().cawn_mixing_bwd(
        ctypes.byref(params), _dp(h), _dp(conv_w), _dp(conv_bias), _dp(gamma), _dp(theta), _dp(saved_states),
        _dp(state_in), _dp(grad_y), _dp(grad_state_out), _dp(grad_h), _dp(grad_conv_w), _dp(grad_conv_bias),
        _dp(grad_gamma), _dp(grad_theta), _dp(grad_state_in), _dp(workspace),
        workspace.numel() * workspace.element_size(), _stream(stream)), "cawn_mixing_bwd")
