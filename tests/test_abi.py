"""The C-ABI library loads on a machine without a GPU, exports every symbol the header
declares, and rejects bad arguments before anything is launched."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2604_04250_b200 import binding as cb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def header_symbols():
    text = open(os.path.join(ROOT, "include", "cawn.h")).read()
    return sorted(set(re.findall(r"CAWN_API\s+[\w\s\*]*?\b(cawn_\w+)\s*\(", text)))


def test_header_and_library_agree():
    syms = header_symbols()
    assert set(syms) == set(cb.EXPORTS)
    lib = ctypes.CDLL(cb.LIB_PATH)
    for s in syms:
        assert hasattr(lib, s), s


def test_params_struct_layout():
    assert ctypes.sizeof(cb.cawn_params) == 48
    assert cb.cawn_params.L.offset == 8 and cb.cawn_params.flags.offset == 44


def test_status_strings():
    assert cb.status_string(0) == "ok"
    assert "carry" in cb.status_string(cb.CAWN_ERR_CARRY_TIMEOUT)
    assert "unknown" in cb.status_string(12345)


def test_workspace_sizes_are_host_only_and_monotone():
    small = cb.cawn_workspace_bytes(cb.make_params(1, 256, 4, 16), cb.CAWN_OP_FWD)
    big = cb.cawn_workspace_bytes(cb.make_params(8, 2048, 12, 64), cb.CAWN_OP_FWD)
    assert 256 < small < big
    # tile = 128 steps, 64-channel groups; per (batch, group): one 64 x 16 B aggregate record per
    # tile (16) plus one checkpoint record per 7 tiles (16 // 7 + 1 = 3 slots)
    assert big == 256 + 8 * 12 * (16 + 3) * 64 * 16
    st = cb.cawn_workspace_bytes(cb.make_params(2, 10, 12, 64, conv_k=4), cb.CAWN_OP_STATE)
    assert st == 2 * 768 * 8 + 2 * 3 * 768 * 4
    saved = cb.cawn_workspace_bytes(cb.make_params(8, 4096, 12, 64), cb.CAWN_OP_BWD_SAVED)
    pushes = cb.cawn_workspace_bytes(cb.make_params(8, 4096, 12, 64), cb.CAWN_OP_BWD_PUSHES)
    assert pushes - saved == 8 * 4096 * 768 * 8


def test_rejections_before_launch():
    lib = cb.lib()
    good = cb.make_params(1, 16, 1, 64)
    n = ctypes.c_size_t()
    bad = cb.make_params(1, 16, 1, 64)
    bad.struct_size = 12
    assert lib.cawn_workspace_bytes(ctypes.byref(bad), 0, ctypes.byref(n)) == cb.CAWN_ERR_INVALID_ARG
    assert lib.cawn_workspace_bytes(ctypes.byref(cb.make_params(0, 16, 1, 64)), 0, ctypes.byref(n)) == cb.CAWN_ERR_INVALID_ARG
    assert lib.cawn_workspace_bytes(ctypes.byref(cb.make_params(1, -1, 1, 64)), 0, ctypes.byref(n)) == cb.CAWN_ERR_INVALID_ARG
    assert lib.cawn_workspace_bytes(ctypes.byref(good), 99, ctypes.byref(n)) == cb.CAWN_ERR_INVALID_ARG
    assert lib.cawn_workspace_bytes(ctypes.byref(good), 0, None) == cb.CAWN_ERR_NULL_POINTER
    assert lib.cawn_workspace_bytes(None, 0, ctypes.byref(n)) == cb.CAWN_ERR_NULL_POINTER
    # forward: NULL and misaligned pointers are caught on the host (fake, never dereferenced, addresses)
    a = 0x10000
    f = lib.cawn_phase_accumulate_fwd
    assert f(ctypes.byref(good), a, None, a, None, None, None, None, None, a, None, None, a, 1 << 20, None) == cb.CAWN_ERR_NULL_POINTER
    assert f(ctypes.byref(good), a + 4, a, a, None, None, None, None, None, a, None, None, a, 1 << 20, None) == cb.CAWN_ERR_MISALIGNED
    assert f(ctypes.byref(good), a, a, a, None, None, None, None, None, a, None, None, a, 16, None) == cb.CAWN_ERR_WORKSPACE_TOO_SMALL
    neg = cb.make_params(1, 16, 1, 64, gate_eps=-1.0)
    assert f(ctypes.byref(neg), a, a, a, None, None, None, None, None, a, None, None, a, 1 << 20, None) == cb.CAWN_ERR_INVALID_ARG
    assert lib.cawn_state_carry(ctypes.byref(good), a, a, -5, a, a, a, None) == cb.CAWN_ERR_INVALID_ARG
    assert lib.cawn_poll_status(None, None) == cb.CAWN_ERR_NULL_POINTER
