"""GPU parity: autoregressive decode, one token per call (L = 1) with the state blob (accumulated
wave state + conv history) carried in place between calls, against one sequential oracle pass.
This is the paper's O(1) generation step: the cost of token 10,000 is that of token 2."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2604_04250_b200 import inputs
from helpers import floored_rel_err

TOL = 1e-4


def test_fused_decode_token_by_token_in_place_state():
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    B, n, C, Kc = 3, 48, 192, 4
    d = inputs.fused_inputs(B, n, C, seed=71, conv_k=Kc, with_bias=True)
    tau = inputs.gate_tau(0.1)
    y_ref, so_ref, m_ref, tail_ref = oracle.fused_forward(d["h"], d["conv_w"], d["gamma"], d["theta"], 0.1, tau,
                                                          bias=d["conv_bias"])
    prm = cb.make_params(B, 1, 3, 64, gate_eps=0.1, gate_tau=float(tau), conv_k=Kc)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    blob, off = state_blob(B, C, Kc)                       # zero state, zero history
    g, t, w, bias = dev(d["gamma"]), dev(d["theta"]), dev(d["conv_w"]), dev(d["conv_bias"])
    h_all = dev(d["h"])
    y = torch.empty((B, 1, C), dtype=torch.complex64, device="cuda")
    ys = []
    for i in range(n):
        cb.cawn_phase_accumulate_fwd(prm, h_all[:, i:i + 1].contiguous(), g, t, y, ws, conv_w=w, conv_bias=bias,
                                     state_in=blob, state_out=blob)
        ys.append(y.clone())
    assert cb.cawn_poll_status(ws) == 0
    got = torch.cat(ys, dim=1).cpu().numpy()
    assert floored_rel_err(got, y_ref, axes=(0, 1)) < TOL
    P, tail = split_blob(blob, off, B, C, Kc)
    assert floored_rel_err(P, so_ref) < TOL
    assert np.array_equal(tail, tail_ref)


def test_cartesian_decode_token_by_token():
    import torch
    from gpu_util import dev
    from paper_2604_04250_b200 import binding as cb
    B, n, C = 2, 40, 768
    d = inputs.scan_inputs(B, n, C, seed=72)
    y_ref, so_ref, _ = oracle.forward(d["p"], d["gamma"], d["theta"], 0.1)
    prm = cb.make_params(B, 1, 12, 64, gate_eps=0.1)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    g, t, p = dev(d["gamma"]), dev(d["theta"]), dev(d["p"])
    state = torch.zeros((B, C), dtype=torch.complex64, device="cuda")
    y = torch.empty((B, n, C), dtype=torch.complex64, device="cuda")
    for i in range(n):
        cb.cawn_phase_accumulate_fwd(prm, p[:, i:i + 1].contiguous(), g, t, y[:, i:i + 1].contiguous(), ws,
                                     state_in=state, state_out=state)
    assert cb.cawn_poll_status(ws) == 0
    assert floored_rel_err(state.cpu().numpy(), so_ref) < TOL


def test_decode_steps_captured_in_a_cuda_graph():
    """The decode loop recorded once into a CUDA graph and replayed: the calls allocate nothing and
    synchronise nothing, and the workspace's epoch protocol needs no reset between replays."""
    import torch
    from gpu_util import dev, state_blob, split_blob
    from paper_2604_04250_b200 import binding as cb
    B, n, C, Kc = 1, 24, 768, 4
    d = inputs.fused_inputs(B, n, C, seed=73, conv_k=Kc)
    tau = inputs.gate_tau(0.1)
    y_ref, so_ref, _, tail_ref = oracle.fused_forward(d["h"], d["conv_w"], d["gamma"], d["theta"], 0.1, tau)
    prm = cb.make_params(B, 1, 12, 64, gate_eps=0.1, gate_tau=float(tau), conv_k=Kc)
    ws = cb.new_workspace(prm, cb.CAWN_OP_FWD)
    blob, off = state_blob(B, C, Kc)
    g, t, w = dev(d["gamma"]), dev(d["theta"]), dev(d["conv_w"])
    rows = [dev(d["h"][:, i:i + 1]) for i in range(n)]
    ys = torch.full((n, B, 1, C), float("nan"), dtype=torch.complex64, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                      # first use outside the capture (one-time kernel attributes)
        cb.cawn_phase_accumulate_fwd(prm, rows[0], g, t, ys[0], ws, conv_w=w, state_in=blob, state_out=blob)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for i in range(n):
            cb.cawn_phase_accumulate_fwd(prm, rows[i], g, t, ys[i], ws, conv_w=w, state_in=blob, state_out=blob)
    for _ in range(2):                                 # two replays from a zero state give the same, right answer
        blob.zero_()
        ys.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert cb.cawn_poll_status(ws) == 0
        got = ys.cpu().numpy()[:, :, 0].transpose(1, 0, 2)
        assert floored_rel_err(got, y_ref, axes=(0, 1)) < TOL
        P, tail = split_blob(blob, off, B, C, Kc)
        assert floored_rel_err(P, so_ref) < TOL
        assert np.array_equal(tail, tail_ref)
