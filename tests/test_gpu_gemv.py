"""The CUDA-core kernel for a handful of rows (M <= 4): every instantiation against the CPU
oracle, bit for bit on integer-valued data (any summation order gives the exact sum there) and
within the tolerance gates on the workloads' own distributions."""
import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt
from test_gpu_parity import run, ternary_case, vid

pytestmark = pytest.mark.gpu

G = kx.KX_PATH_GEMV
GEMV_VARIANTS = [dict(path=G, block_n=rw, split_k=w) for rw in (1, 2, 4) for w in (1, 5, 16)]


@pytest.mark.parametrize("ov", GEMV_VARIANTS, ids=vid)
@pytest.mark.parametrize("N,K", [(8, 8), (264, 72), (1000, 1096), (2048, 4096), (520, 14336)])
def test_gemv_exact_integer_arithmetic(ov, N, K):
    for M in (1, 2, 3, 4):
        X, W, b, R = ternary_case(M, N, K, seed=40 + M)
        ref = oracle.outproj(X, W, b, R)
        y = run(X, W, b, R, ov)
        ok, msg = kt.gate_exact(y, ref)
        assert ok, f"M={M}: {msg}"
        assert np.array_equal(run(X, W, b, R.copy(), ov, inplace=True), y), f"M={M}: in place differs"
    ok, msg = kt.gate_exact(run(X, W, None, None, ov), oracle.outproj(X, W))
    assert ok, msg


def test_gemv_is_the_automatic_plan_for_a_few_rows():
    for M in (1, 4):
        info = kx.kx_plan_query(M, 4096, 4096)
        assert info.path == G and info.grid * info.block_n == 4096 and info.workspace_bytes == 0
    assert kx.kx_plan_query(5, 4096, 4096).path == kx.KX_PATH_SKINNY
    assert kx.kx_plan_query(33, 4096, 4096).path == kx.KX_PATH_SWAP
    assert kx.kx_plan_query(32, 8192, 8192).path == kx.KX_PATH_SWAP      # large W: the split-K tensor-memory kernel
    for bad in (dict(path=G, block_n=3), dict(path=G, split_k=17), dict(path=G, cta_pair=2), dict(path=G, max_ctas=7)):
        with pytest.raises(kx.KxError):
            kx.kx_plan_query(1, 4096, 4096, ov=kx.make_override(**bad))
    with pytest.raises(kx.KxError):
        kx.kx_plan_query(5, 4096, 4096, ov=kx.make_override(path=G))


@pytest.mark.parametrize("ov", [None] + GEMV_VARIANTS[1:4], ids=lambda v: "auto" if v is None else vid(v))
@pytest.mark.parametrize("stress", [False, True], ids=["literal", "stress"])
def test_gemv_random_workloads_all_gates(ov, stress):
    for name, M in (("sweep_M1_H2048", 1), ("sweep_M1_H5120", 1), ("sweep_M1_H4096", 3)):
        wl = inputs.all_workloads()[name]
        d = inputs.make_inputs(wl, stress=stress, M=M)
        ref, absref = oracle.outproj(d["X"], d["W"], d["bias"], d["R"], want_abs=True)
        y = run(d["X"], d["W"], d["bias"], d["R"], ov)
        ok, msg = kt.gate_a(y, ref)
        assert ok, msg
        ok, msg = kt.gate_c(y, ref, absref, wl.K, rate_limit=3e-2 if stress else 5e-3)
        assert ok, msg
        assert np.array_equal(run(d["X"], d["W"], d["bias"], d["R"], ov), y)      # fixed summation order


def test_gemv_zero_weight_selectors_and_scaling():
    M, N, K = 3, 392, 448
    d = inputs.make_inputs(inputs.Workload("t", M, N, K, 33, True, True), stress=True)
    W0 = np.zeros((N, K), dtype=np.uint16)
    assert np.array_equal(run(d["X"], W0, None, d["R"]), d["R"])
    f = oracle.widen_bf16
    assert np.array_equal(run(d["X"], W0, d["bias"], d["R"]), oracle.round_bf16(f(d["R"]) + f(d["bias"])[None, :]))
    W, pi = inputs.permutation_matrix_bf16(5, N, K)
    X = inputs.normal_bf16(5, "X", (M, K), 1.0)
    assert np.array_equal(run(X, W, None, None), X[:, pi])
    X1 = inputs.one_hot_rows_bf16(M, K)
    Wr = inputs.normal_bf16(6, "W", (N, K), 1.0)
    assert np.array_equal(run(X1, Wr, None, None), Wr[:, np.arange(M) % K].T)
    y1 = run(d["X"], d["W"], None, None)
    X2 = inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(d["X"]))
    assert np.array_equal(run(X2, d["W"], None, None), inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(y1)))


@pytest.mark.parametrize("depth", [-1, 0, 1, 1000])
def test_gemv_l2_request_is_a_hint_and_rewritten_operands_are_seen(depth):
    """The rows requested into L2 before the dependency wait change no bit, and W / X rewritten by the
    kernel just before this one in the stream (whose tail the prologue overlaps) are read fresh."""
    import torch
    M, N, K = 2, 520, 1096
    X, W, b, R = ternary_case(M, N, K, seed=35)
    ov = dict(path=G, block_n=2, split_k=4, l2_prefetch=depth)
    y = run(X, W, b, R, ov)
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg
    tX2, tR, tb, tW2 = kt.to_dev(X), kt.to_dev(R), kt.to_dev(b), kt.to_dev(W)
    tW, tX = torch.zeros_like(tW2), torch.zeros_like(tX2)
    eye = torch.eye(K, dtype=torch.bfloat16, device="cuda")
    tY = kt.nan_filled(M, N)
    o = kx.make_override(**ov)
    for _ in range(3):
        tW.zero_(); tX.zero_()
        kx.kx_gemm_bf16(tX2, eye, tX)
        kx.kx_gemm_bf16(tW2, eye, tW)
        kx.kx_outproj_residual_ex(tX, tW, tb, tR, tY, o)
    assert np.array_equal(kt.from_dev(tY), y)


def test_gemv_pitched_operands_and_canaries():
    import torch
    M, N, K = 4, 264, 520
    X, W, b, R = ternary_case(M, N, K, seed=37)
    ref = oracle.outproj(X, W, b, R)
    ldx, ldw, ldr, ldy = K + 24, K + 8, N + 16, N + 40
    def pitched(a, ld):
        t = torch.full((a.shape[0], ld), float("nan"), dtype=torch.bfloat16, device="cuda")
        t[:, :a.shape[1]] = kt.to_dev(a)
        return t
    tX, tW, tR = pitched(X, ldx), pitched(W, ldw), pitched(R, ldr)
    tY = torch.full((M, ldy), -7.0, dtype=torch.bfloat16, device="cuda")
    kx.kx_outproj_residual_strided(tX[:, :K], tW[:, :K], kt.to_dev(b), tR[:, :N], tY[:, :N])
    torch.cuda.synchronize()
    ok, msg = kt.gate_exact(kt.from_dev(tY[:, :N].contiguous()), ref)
    assert ok, msg
    assert (tY[:, N:] == -7.0).all()


# ------------------------------------------------------------------ 5..32 rows: warp-level tensor-core kernel
K4 = kx.KX_PATH_SKINNY
SKINNY_VARIANTS = [dict(path=K4, block_n=16), dict(path=K4, block_n=32)]


@pytest.mark.parametrize("ov", SKINNY_VARIANTS, ids=vid)
@pytest.mark.parametrize("N,K", [(8, 8), (264, 72), (1000, 1096), (2048, 4096), (520, 14336)])
def test_skinny_exact_integer_arithmetic(ov, N, K):
    for M in (1, 5, 8, 9, 16, 23, 32):
        X, W, b, R = ternary_case(M, N, K, seed=60 + M)
        ref = oracle.outproj(X, W, b, R)
        y = run(X, W, b, R, ov)
        ok, msg = kt.gate_exact(y, ref)
        assert ok, f"M={M}: {msg}"
        assert np.array_equal(run(X, W, b, R.copy(), ov, inplace=True), y), f"M={M}: in place differs"
    ok, msg = kt.gate_exact(run(X, W, None, None, ov), oracle.outproj(X, W))
    assert ok, msg


@pytest.mark.parametrize("ov", SKINNY_VARIANTS, ids=vid)
@pytest.mark.parametrize("stress", [False, True], ids=["literal", "stress"])
def test_skinny_random_workloads_all_gates(ov, stress):
    for name, M in (("sweep_M32_H2048", 32), ("sweep_M32_H5120", 32), ("sweep_M32_H4096", 13)):
        wl = inputs.all_workloads()[name]
        d = inputs.make_inputs(wl, stress=stress, M=M)
        ref, absref = oracle.outproj(d["X"], d["W"], d["bias"], d["R"], want_abs=True)
        y = run(d["X"], d["W"], d["bias"], d["R"], ov)
        ok, msg = kt.gate_a(y, ref)
        assert ok, msg
        ok, msg = kt.gate_c(y, ref, absref, wl.K, rate_limit=3e-2 if stress else 5e-3)
        assert ok, msg
        assert np.array_equal(run(d["X"], d["W"], d["bias"], d["R"], ov), y)      # fixed summation order


@pytest.mark.parametrize("ov", SKINNY_VARIANTS, ids=vid)
def test_skinny_zero_weight_selectors_scaling_and_plain_gemm(ov):
    M, N, K = 27, 392, 448
    d = inputs.make_inputs(inputs.Workload("t", M, N, K, 34, True, True), stress=True)
    W0 = np.zeros((N, K), dtype=np.uint16)
    assert np.array_equal(run(d["X"], W0, None, d["R"], ov), d["R"])
    f = oracle.widen_bf16
    assert np.array_equal(run(d["X"], W0, d["bias"], d["R"], ov), oracle.round_bf16(f(d["R"]) + f(d["bias"])[None, :]))
    W, pi = inputs.permutation_matrix_bf16(5, N, K)
    X = inputs.normal_bf16(5, "X", (M, K), 1.0)
    assert np.array_equal(run(X, W, None, None, ov), X[:, pi])
    X1 = inputs.one_hot_rows_bf16(M, K)
    Wr = inputs.normal_bf16(6, "W", (N, K), 1.0)
    assert np.array_equal(run(X1, Wr, None, None, ov), Wr[:, np.arange(M) % K].T)
    y1 = run(d["X"], d["W"], None, None, ov)
    X2 = inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(d["X"]))
    assert np.array_equal(run(X2, d["W"], None, None, ov), inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(y1)))
    wl = inputs.all_workloads()["cfg4"]
    dd = inputs.make_inputs(wl, M=30, N=1040, K=2048)
    assert kt.rel_fro(run(dd["X"], dd["W"], None, None, ov), oracle.outproj(dd["X"], dd["W"])) <= 2.0 ** -8


@pytest.mark.parametrize("depth", [-1, 0, 1, 1000])
def test_skinny_l2_request_is_a_hint_and_rewritten_operands_are_seen(depth):
    import torch
    M, N, K = 19, 520, 1096
    X, W, b, R = ternary_case(M, N, K, seed=36)
    ov = dict(path=K4, block_n=32, l2_prefetch=depth)
    y = run(X, W, b, R, ov)
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg
    tX2, tR, tb, tW2 = kt.to_dev(X), kt.to_dev(R), kt.to_dev(b), kt.to_dev(W)
    tW, tX = torch.zeros_like(tW2), torch.zeros_like(tX2)
    eye = torch.eye(K, dtype=torch.bfloat16, device="cuda")
    tY = kt.nan_filled(M, N)
    o = kx.make_override(**ov)
    for _ in range(3):
        tW.zero_(); tX.zero_()
        kx.kx_gemm_bf16(tX2, eye, tX)
        kx.kx_gemm_bf16(tW2, eye, tW)
        kx.kx_outproj_residual_ex(tX, tW, tb, tR, tY, o)
    assert np.array_equal(kt.from_dev(tY), y)


def test_skinny_pitched_operands_special_values_and_canaries():
    import torch
    M, N, K = 21, 264, 520
    X, W, b, R = ternary_case(M, N, K, seed=38)
    X = X.copy(); R = R.copy()
    X[5, 70] = 0x7F80          # +inf in one row of X
    X[10, 3] = 0x7FC0          # NaN in another
    R[17, 200] = 0xFF80        # -inf in one residual element
    ref = oracle.outproj(X, W, b, R)
    ldx, ldw, ldr, ldy = K + 24, K + 8, N + 16, N + 40
    def pitched(a, ld):
        t = torch.full((a.shape[0], ld), float("nan"), dtype=torch.bfloat16, device="cuda")
        t[:, :a.shape[1]] = kt.to_dev(a)
        return t
    tX, tW, tR = pitched(X, ldx), pitched(W, ldw), pitched(R, ldr)
    tY = torch.full((M, ldy), -7.0, dtype=torch.bfloat16, device="cuda")
    kx.kx_outproj_residual_strided(tX[:, :K], tW[:, :K], kt.to_dev(b), tR[:, :N], tY[:, :N])
    torch.cuda.synchronize()
    y = oracle.widen_bf16(kt.from_dev(tY[:, :N].contiguous()))
    assert np.array_equal(np.isnan(y), np.isnan(ref))
    fin = np.isfinite(ref)
    assert np.array_equal(oracle.round_bf16(ref[fin]), oracle.round_bf16(y[fin]))
    assert np.isnan(y[10]).all() and y[17, 200] == -np.inf
    assert (tY[:, N:] == -7.0).all()
