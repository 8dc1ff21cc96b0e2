"""After kx_init the device entry points neither allocate nor synchronise, so a sequence of
calls can be captured into a CUDA graph and replayed (cluster launches and programmatic
dependent launch included).  Replays must reproduce the eager results bit for bit."""
import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu


def test_capture_and_replay_a_layer_tail():
    import torch
    kx.kx_init(torch.cuda.current_device())
    M, N, K, I = 384, 1024, 1024, 1536
    d = inputs.make_inputs(inputs.Workload("t", M, N, K, 501, True, True), stress=True)
    g = inputs.normal_bf16(501, "X", (N,), 1.0)
    Wg = inputs.normal_bf16(502, "W", (I, N), 1.0 / np.sqrt(N))
    Wu = inputs.normal_bf16(503, "W", (I, N), 1.0 / np.sqrt(N))
    X, W, b, R = (kt.to_dev(d[k]) for k in ("X", "W", "bias", "R"))
    gd, Wgd, Wud = kt.to_dev(g), kt.to_dev(Wg), kt.to_dev(Wu)
    Xs = kt.to_dev(d["X"][:8].copy())            # a small-M call (cluster split-K path) in the same graph
    Rs = kt.to_dev(d["R"][:8].copy())

    def layer(H, Z, A, Ysmall):
        kx.kx_outproj_residual_rmsnorm(X, W, b, R, gd, 1e-6, H, Z)   # projection + residual, RMSNorm
        kx.kx_gate_up_swiglu(Z, Wgd, Wud, A)                          # gate/up + SwiGLU
        kx.kx_outproj_residual(Xs, W, b, Rs, Ysmall)                  # small-M path

    eager = [kt.nan_filled(M, N), kt.nan_filled(M, N), kt.nan_filled(M, I), kt.nan_filled(8, N)]
    layer(*eager)
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    want = [kt.from_dev(t) for t in eager]

    outs = [kt.nan_filled(M, N), kt.nan_filled(M, N), kt.nan_filled(M, I), kt.nan_filled(8, N)]
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        layer(*outs)                                  # warm-up on the side stream
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=s):
            layer(*outs)
    for rep in range(3):
        for t in outs:
            t.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert kx.kx_last_device_status()[0] == kx.KX_OK
        for got, ref in zip(outs, want):
            assert np.array_equal(kt.from_dev(got), ref)
    # and the captured results are right, not merely reproducible
    ok, msg = kt.gate_a(want[0], oracle.outproj(d["X"], d["W"], d["bias"], d["R"]))
    assert ok, msg
    ok, msg = kt.gate_a(want[2], oracle.swiglu(want[1], Wg, Wu))
    assert ok, msg
