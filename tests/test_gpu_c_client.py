"""GPU: the C ABI used from a plain C program (no Python or PyTorch in the process): compile
tests/c_client/cawn_client.c against include/cawn.h and libcawn.so, run it on files of seeded inputs,
and compare what it writes with the oracle."""
import os
import shutil
import subprocess

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import binding as cb, inputs
from helpers import floored_rel_err, unpack_mask

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)


def test_plain_c_client_forward_and_backward(tmp_path):
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    gcc = shutil.which("gcc")
    if gcc is None or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime.h")):
        pytest.skip("no host C compiler or CUDA runtime headers")
    cb.lib()                                                 # makes sure the library is built
    exe = str(tmp_path / "cawn_client")
    libdir = os.path.dirname(cb.LIB_PATH)
    subprocess.check_call([gcc, "-O1", "-std=c11", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                           os.path.join(HERE, "c_client", "cawn_client.c"), "-o", exe,
                           "-L", libdir, "-l:libcawn.so", "-L", os.path.join(cuda, "lib64"), "-lcudart",
                           "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    B, L, H, F = 2, 700, 3, 64
    C = H * F
    d = inputs.scan_inputs(B, L, C, seed=2100, with_state=True, with_grad=True)
    eps = 0.1
    fin, fout = str(tmp_path / "in.bin"), str(tmp_path / "out.bin")
    with open(fin, "wb") as f:
        np.array([B, L, H, F], np.int32).tofile(f)
        np.array([eps], np.float32).tofile(f)
        for a in (d["p"], d["gamma"], d["theta"], d["state_in"], d["grad_y"]):
            np.ascontiguousarray(a).tofile(f)
    out = subprocess.run([exe, fin, fout], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    raw = np.fromfile(fout, np.uint8)
    n, MW = B * L * C, (C + 31) // 32
    sizes = [n * 8, B * C * 8, B * L * MW * 4, n * 8, C * 4, C * 4, B * C * 8]
    assert raw.size == sum(sizes)
    parts = np.split(raw, np.cumsum(sizes)[:-1])
    y = parts[0].view(np.complex64).reshape(B, L, C)
    so = parts[1].view(np.complex64).reshape(B, C)
    mask = parts[2].view(np.uint32).reshape(B, L, MW)
    gp = parts[3].view(np.complex64).reshape(B, L, C)
    gg, gt = parts[4].view(np.float32), parts[5].view(np.float32)
    gsi = parts[6].view(np.complex64).reshape(B, C)
    si = d["state_in"].astype(np.complex128)
    y_ref, so_ref, m_ref = oracle.forward(d["p"], d["gamma"], d["theta"], eps, state_in=si)
    assert floored_rel_err(y, y_ref, axes=(0, 1)) < 1e-4
    assert floored_rel_err(so, so_ref) < 1e-4
    assert np.array_equal(unpack_mask(mask, C), m_ref)
    z, _ = oracle.gate(d["p"], eps)
    ref = oracle.scan_bwd(z, d["theta"], d["grad_y"], gamma=d["gamma"], state_in=si)
    assert floored_rel_err(gp, ref["dp"], axes=(0, 1)) < 1e-4
    assert floored_rel_err(gg, ref["dgamma"]) < 1e-4
    assert floored_rel_err(gt, ref["dtheta"]) < 1e-4
    assert floored_rel_err(gsi, ref["dstate_in"]) < 1e-4
