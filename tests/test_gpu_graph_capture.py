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


def test_capture_and_replay_the_int8_branch():
    """RMSNorm + code book -> weights' code books -> INT8 gate/up + SwiGLU -> FP8 projection, captured
    and replayed: same bits as the eager run."""
    import torch
    kx.kx_init(torch.cuda.current_device())
    M, N, I = 384, 1024, 1536
    H = kt.to_dev(inputs.normal_bf16(511, "R", (M, N), 1.0))
    g = kt.to_dev(inputs.normal_bf16(511, "bias", (N,), 1.0))
    Wg = kt.to_dev(inputs.normal_bf16(512, "W", (I, N), 1.0 / np.sqrt(N)))
    Wu = kt.to_dev(inputs.normal_bf16(513, "W", (I, N), 1.0 / np.sqrt(N)))
    i8 = lambda *shape: torch.zeros(shape, dtype=torch.int8, device="cuda")
    f32 = lambda n: torch.zeros((n,), dtype=torch.float32, device="cuda")
    f8 = lambda *shape: torch.zeros(shape, dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn)

    def branch(Xq, sx, Qg, Sg, Qu, Su, Z, X8, s8, W8, sw8, Y):
        kx.kx_rmsnorm_quantize_int8(H, g, 1e-6, Xq, sx)
        kx.kx_quantize_gate_up_int8(Wg, Wu, Qg, Sg, Qu, Su)
        kx.kx_gate_up_swiglu_int8(Xq, sx, Qg, Sg, Qu, Su, Z)
        kx.kx_rmsnorm_quantize_fp8(H, g, 1e-6, X8, s8)
        kx.kx_quantize_rows_fp8(Wg, W8, sw8)
        kx.kx_outproj_residual_fp8(X8, s8, W8, sw8, None, None, Y)

    def bufs():
        return [i8(M, N), f32(M), i8(I, N), f32(I), i8(I, N), f32(I), kt.nan_filled(M, I),
                f8(M, N), f32(M), f8(I, N), f32(I), kt.nan_filled(M, I)]

    raw = lambda t: t.view(torch.uint8).cpu().numpy() if t.dtype not in (torch.float32, torch.bfloat16) else (
        t.cpu().numpy() if t.dtype == torch.float32 else kt.from_dev(t))
    eager = bufs()
    branch(*eager)
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    want = [raw(t) for t in eager]
    outs = bufs()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        branch(*outs)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=s):
            branch(*outs)
    for rep in range(2):
        for t in outs:
            t.view(torch.uint8).zero_() if t.dtype not in (torch.float32, torch.bfloat16) else t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert kx.kx_last_device_status()[0] == kx.KX_OK
        for got, ref in zip(outs, want):
            assert np.array_equal(raw(got), ref)
    ok, msg = kt.gate_a(want[6], oracle.swiglu_int8(want[0].view(np.int8), want[1], want[2].view(np.int8), want[3],
                                                    want[4].view(np.int8), want[5]))
    assert ok, msg
    ok, msg = kt.gate_a(want[11], oracle.outproj_fp8(want[7], want[8], want[9], want[10]))
    assert ok, msg


def test_capture_and_replay_the_block_scaled_branch():
    """RMSNorm + block-scaled code book -> weights' code book -> block-scaled projection with residual,
    captured and replayed: same bits as the eager run (no allocation or host work in the calls)."""
    import torch
    kx.kx_init(torch.cuda.current_device())
    M, N, K = 384, 1160, 1024
    H = kt.to_dev(inputs.normal_bf16(521, "R", (M, K), 1.0))
    g = kt.to_dev(inputs.normal_bf16(521, "bias", (K,), 1.0))
    W = kt.to_dev(inputs.normal_bf16(522, "W", (N, K), 1.0 / np.sqrt(K)))
    R = kt.to_dev(inputs.normal_bf16(523, "R", (M, N), 1.0))
    f8 = lambda *shape: torch.zeros(shape, dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn)
    u8 = lambda n: torch.zeros((n,), dtype=torch.uint8, device="cuda")

    def branch(Xq, SFX, Wq, SFW, Y):
        kx.kx_rmsnorm_quantize_mxfp8(H, g, 1e-6, Xq, SFX)
        kx.kx_quantize_rows_mxfp8(W, Wq, SFW)
        kx.kx_outproj_residual_mxfp8(Xq, SFX, Wq, SFW, None, R, Y)

    def bufs():
        return [f8(M, K), u8(kx.kx_mx_scale_bytes(M, K)), f8(N, K), u8(kx.kx_mx_scale_bytes(N, K)), kt.nan_filled(M, N)]

    raw = lambda t: kt.from_dev(t) if t.dtype == torch.bfloat16 else t.view(torch.uint8).cpu().numpy()
    eager = bufs()
    branch(*eager)
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    want = [raw(t) for t in eager]
    outs = bufs()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        branch(*outs)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=s):
            branch(*outs)
    for rep in range(2):
        for t in outs:
            t.zero_() if t.dtype == torch.bfloat16 else t.view(torch.uint8).zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert kx.kx_last_device_status()[0] == kx.KX_OK
        for got, ref in zip(outs, want):
            assert np.array_equal(raw(got), ref)


def test_capture_and_replay_the_4bit_branch():
    """4-bit code books -> 4-bit block-scaled projection with residual, captured and replayed: same bits."""
    import torch
    kx.kx_init(torch.cuda.current_device())
    M, N, K = 384, 1160, 1024
    X = kt.to_dev(inputs.normal_bf16(531, "X", (M, K), 1.0))
    W = kt.to_dev(inputs.normal_bf16(532, "W", (N, K), 1.0 / np.sqrt(K)))
    R = kt.to_dev(inputs.normal_bf16(533, "R", (M, N), 1.0))
    gsx, gsw = 6.0 / 2688.0, 0.2 / 2688.0
    u8 = lambda *shape: torch.zeros(shape, dtype=torch.uint8, device="cuda")

    def branch(Xq, SFX, Wq, SFW, Y):
        kx.kx_quantize_rows_nvfp4(X, gsx, Xq, SFX)
        kx.kx_quantize_rows_nvfp4(W, gsw, Wq, SFW)
        kx.kx_outproj_residual_nvfp4(Xq, SFX, Wq, SFW, gsx * gsw, None, R, Y)

    def bufs():
        return [u8(M, K // 2), u8(kx.kx_nvfp4_scale_bytes(M, K)), u8(N, K // 2), u8(kx.kx_nvfp4_scale_bytes(N, K)),
                kt.nan_filled(M, N)]

    raw = lambda t: kt.from_dev(t) if t.dtype == torch.bfloat16 else t.cpu().numpy()
    eager = bufs()
    branch(*eager)
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    want = [raw(t) for t in eager]
    assert want[0].any() and not np.isnan(oracle.widen_bf16(want[4])).any()
    outs = bufs()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        branch(*outs)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=s):
            branch(*outs)
    for rep in range(2):
        for t in outs:
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert kx.kx_last_device_status()[0] == kx.KX_OK
        for got, ref in zip(outs, want):
            assert np.array_equal(raw(got), ref)
