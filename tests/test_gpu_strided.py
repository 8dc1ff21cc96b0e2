"""Row-pitched operands: slices of wider buffers go through the same kernels (tensor-map row
strides), on every path, and give exactly the bits of the dense call on packed copies."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu


def wide(bits, ld, pad_value=0x7FC0):
    """Device buffer [rows, ld] pre-filled with NaN patterns; the matrix sits in the left columns."""
    rows, cols = bits.shape
    buf = torch.full((rows, ld), 0, dtype=torch.int16, device="cuda")
    buf.fill_(np.int16(pad_value).item() if pad_value < 0x8000 else pad_value - 0x10000)
    buf[:, :cols] = torch.from_numpy(bits.view(np.int16)).cuda()
    return buf.view(torch.bfloat16)


# small-M path (cluster and workspace split-K), single-CTA tiles, K cluster, CTA pairs with a half-width tail and
# (last shape: 110 pair tiles of 192 columns on 74 slots, 64 k-blocks) with a K-halves tail
@pytest.mark.parametrize("M,N,K", [(1, 520, 1096), (37, 2048, 2048), (200, 1024, 4096), (300, 520, 264), (512, 2048, 2048),
                                   (1000, 776, 1096), (2381, 4096, 512), (2560, 2048, 4096)])
def test_strided_equals_dense(M, N, K):
    d = inputs.make_inputs(inputs.Workload("t", M, N, K, 900 + M, True, True), stress=True)
    Yd = kt.nan_filled(M, N)
    kx.kx_outproj_residual(kt.to_dev(d["X"]), kt.to_dev(d["W"]), kt.to_dev(d["bias"]), kt.to_dev(d["R"]), Yd)
    want = kt.from_dev(Yd)
    ok, msg = kt.gate_a(want, oracle.outproj(d["X"], d["W"], d["bias"], d["R"]))
    assert ok, msg
    ldx, ldw, ldr, ldy = K + 64, K + 8, N + 24, N + 40
    Xw, Ww, Rw = wide(d["X"], ldx), wide(d["W"], ldw), wide(d["R"], ldr)
    Yw = torch.full((M, ldy), 0, dtype=torch.int16, device="cuda")
    Yw.fill_(0x1234)
    Yw = Yw.view(torch.bfloat16)
    kx.kx_outproj_residual_strided(Xw[:, :K], Ww[:, :K], kt.to_dev(d["bias"]), Rw[:, :N], Yw[:, :N])
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    got = Yw.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got[:, :N], want)
    assert (got[:, N:] == 0x1234).all()                      # the padding of Y is never written
    # in place on a pitched residual stream, and without bias / residual
    Rw2 = wide(d["R"], ldr, pad_value=0x1234)
    kx.kx_outproj_residual_strided(Xw[:, :K], Ww[:, :K], kt.to_dev(d["bias"]), Rw2[:, :N], Rw2[:, :N])
    got2 = Rw2.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got2[:, :N], want) and (got2[:, N:] == 0x1234).all()
    Yp = kt.nan_filled(M, N)
    kx.kx_gemm_bf16(kt.to_dev(d["X"]), kt.to_dev(d["W"]), Yp)
    kx.kx_outproj_residual_strided(Xw[:, :K], Ww[:, :K], None, None, Yw[:, :N])
    assert np.array_equal(Yw.view(torch.int16).cpu().numpy().view(np.uint16)[:, :N], kt.from_dev(Yp))


@pytest.mark.parametrize("M,N,K", [(5, 264, 100), (300, 520, 77), (700, 1024, 1001), (64, 128, 1), (130, 256, 63)])
def test_any_reduction_length_with_padded_rows(M, N, K):
    """K that is not a multiple of 8 (nor of the 64-wide k-block): rows padded to a multiple of 8; whatever
    sits in the padding (NaN here) must not reach the result.  Ternary data: bit-exact."""
    X = inputs.ternary_bf16(910, "X", (M, K))
    W = inputs.ternary_bf16(910, "W", (N, K))
    b = inputs.small_int_bf16(910, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(910, "R", (M, N), -8, 8)
    ld = (K + 7) // 8 * 8 + 8
    Y = kt.nan_filled(M, N)
    kx.kx_outproj_residual_strided(wide(X, ld)[:, :K], wide(W, ld)[:, :K], kt.to_dev(b), kt.to_dev(R), Y)
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    ok, msg = kt.gate_exact(kt.from_dev(Y), oracle.outproj(X, W, b, R))
    assert ok, msg


@pytest.mark.parametrize("M,N,K", [(5, 61, 100), (300, 517, 77), (700, 1001, 1001), (64, 130, 1), (130, 255, 63), (2381, 1003, 520)])
def test_any_output_width_with_padded_rows(M, N, K):
    """N that is not a multiple of 8: pitched Y / R, the last columns clipped by the TMA store, the bias
    tail added element by element; nothing beyond the 16-byte unit that holds column N - 1 is written.  Ternary
    data: bit-exact."""
    X = inputs.ternary_bf16(915, "X", (M, K))
    W = inputs.ternary_bf16(915, "W", (N, K))
    b = inputs.small_int_bf16(915, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(915, "R", (M, N), -8, 8)
    ldk = (K + 7) // 8 * 8 + 8
    ldn = (N + 7) // 8 * 8 + 8
    Yw = torch.zeros((M, ldn), dtype=torch.int16, device="cuda")
    Yw.fill_(0x1234)
    Yw = Yw.view(torch.bfloat16)
    bd = torch.zeros(ldn, dtype=torch.bfloat16, device="cuda")          # bias in an aligned, longer buffer
    bd[:N] = kt.to_dev(b)
    Xw, Ww, Rw = wide(X, ldk), wide(W, ldk), wide(R, ldn)              # keep the buffers alive across the call
    rc = kx.load().kx_outproj_residual_strided(Xw.data_ptr(), ldk, Ww.data_ptr(), ldk, bd.data_ptr(),
                                               Rw.data_ptr(), ldn, Yw.data_ptr(), ldn, M, N, K, None)
    torch.cuda.synchronize()
    assert rc == kx.KX_OK and kx.kx_last_device_status()[0] == kx.KX_OK
    got = Yw.view(torch.int16).cpu().numpy().view(np.uint16)
    ok, msg = kt.gate_exact(got[:, :N], oracle.outproj(X, W, b, R))
    assert ok, msg
    n8 = (N + 7) // 8 * 8            # the store works in 16-byte units: the row's padding up to there may be written
    assert (got[:, n8:] == 0x1234).all()


def test_strided_argument_checks():
    lib = kx.load()
    A = 0x100000
    call = lambda ldx, ldw, ldr, ldy, R=3 * A, Y=4 * A, N=64, K=64: lib.kx_outproj_residual_strided(
        A, ldx, 2 * A, ldw, None, R, ldr, Y, ldy, 16, N, K, None)
    assert call(56, 64, 64, 64) == kx.KX_ERR_SHAPE            # pitch shorter than the row
    assert call(64, 64, 64, 60) == kx.KX_ERR_SHAPE
    assert call(68, 64, 64, 64) == kx.KX_ERR_SHAPE            # pitch not a multiple of 8
    assert call(64, 64, 64, 72, R=4 * A) == kx.KX_ERR_OVERLAP  # in place needs equal pitches
    assert call(64, 64, 64, 64, Y=A + 32) == kx.KX_ERR_OVERLAP
    assert call(64, 64, 64, 64, Y=4 * A + 2) == kx.KX_ERR_ALIGN
    assert lib.kx_outproj_residual_strided(A, 64, 2 * A, 64, None, None, 0, 4 * A, 64, 0, 64, 64, None) == kx.KX_OK
    # K == 0 on pitched buffers: Y = R + bias
    R = inputs.small_int_bf16(920, "R", (6, 16), -8, 8)
    Rw = wide(R, 40)
    Yw = torch.zeros((6, 24), dtype=torch.bfloat16, device="cuda")
    rc = lib.kx_outproj_residual_strided(None, 8, None, 8, None, Rw.data_ptr(), 40, Yw.data_ptr(), 24, 6, 16, 0, None)
    torch.cuda.synchronize()
    assert rc == kx.KX_OK
    assert np.array_equal(Yw.view(torch.int16).cpu().numpy().view(np.uint16)[:, :16], R)


@pytest.mark.parametrize("B,M,N,K,shared", [(3, 200, 520, 264, True), (4, 37, 1024, 1024, False), (2, 1000, 776, 1096, False)])
def test_batched_equals_a_loop_of_single_calls(B, M, N, K, shared):
    """The batched entry point is a loop of ordinary calls: the same bits as calling them one by one,
    with shared or per-problem weights and bias, in place as well."""
    ds = [inputs.make_inputs(inputs.Workload("t", M, N, K, 930 + b, True, True), stress=True) for b in range(B)]
    X = torch.stack([kt.to_dev(d["X"]) for d in ds])
    R = torch.stack([kt.to_dev(d["R"]) for d in ds])
    W = kt.to_dev(ds[0]["W"]) if shared else torch.stack([kt.to_dev(d["W"]) for d in ds])
    bias = kt.to_dev(ds[0]["bias"]) if shared else torch.stack([kt.to_dev(d["bias"]) for d in ds])
    Y = torch.full((B, M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    kx.kx_outproj_residual_batched(X, W, bias, R, Y)
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    for b in range(B):
        Yb = kt.nan_filled(M, N)
        kx.kx_outproj_residual(X[b], W if shared else W[b], bias if shared else bias[b], R[b], Yb)
        assert np.array_equal(kt.from_dev(Y[b].contiguous()), kt.from_dev(Yb))
    d = ds[B - 1]
    ok, msg = kt.gate_a(kt.from_dev(Y[B - 1].contiguous()), oracle.outproj(d["X"], ds[0]["W"] if shared else d["W"],
                                                                            ds[0]["bias"] if shared else d["bias"], d["R"]))
    assert ok, msg
    want = kt.from_dev(Y.reshape(B * M, N))
    Rc = R.clone()
    kx.kx_outproj_residual_batched(X, W, bias, Rc, Rc)                      # in place
    assert np.array_equal(kt.from_dev(Rc.reshape(B * M, N)), want)
    lib = kx.load()
    A = 0x100000
    assert lib.kx_outproj_residual_batched(A, 64 * 16, 2 * A, 0, None, 0, None, 0, 4 * A, 16 * 8, 16, 64, 64, 2, None) == kx.KX_ERR_OVERLAP
    assert lib.kx_outproj_residual_batched(A, 64 * 16 + 4, 2 * A, 0, None, 0, None, 0, 4 * A, 16 * 64, 16, 64, 64, 2, None) == kx.KX_ERR_ALIGN
    assert lib.kx_outproj_residual_batched(A, 0, 2 * A, 0, None, 0, None, 0, 4 * A, 0, 16, 64, 64, 0, None) == kx.KX_OK
