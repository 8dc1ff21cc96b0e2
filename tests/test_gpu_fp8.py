"""FP8 (E4M3) twins of the INT8 branch: code books bit for bit, the FP8 GEMMs bit for bit where
every partial sum is exactly representable, the rest within the tolerance gates of the BF16 path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu

F8 = torch.float8_e4m3fn


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev8(codes):
    return torch.from_numpy(np.ascontiguousarray(codes)).cuda().view(F8)


def host8(t):
    return t.view(torch.uint8).cpu().numpy()


def status_ok():
    code, detail = kx.kx_last_device_status()
    assert code == kx.KX_OK, (code, detail)


# ------------------------------------------------------------------ code books
def gpu_quantize(A):
    rows, cols = A.shape
    Q = torch.full((rows, cols), 0x55, dtype=torch.uint8, device="cuda").view(F8)
    S = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda")
    kx.kx_quantize_rows_fp8(kt.to_dev(A), Q, S)
    return host8(Q), S.cpu().numpy()


@pytest.mark.parametrize("rows,cols", [(1, 16), (5, 48), (300, 2064), (129, 4096), (3, 32768), (700, 1024), (7, 3072), (5, 2560), (9, 7168), (5, 6144), (9000, 256)])
def test_fp8_code_book_bit_exact(rows, cols):
    A = inputs.normal_bf16(700 + cols, "X", (rows, cols), 2.5)
    if rows > 2:
        A[1] = 0
        A[2, : cols // 2] = 0
    Q, S = gpu_quantize(A)
    Qr, Sr = oracle.quantize_rows_fp8(A)
    assert np.array_equal(S.view(np.uint32), Sr.view(np.uint32))
    assert np.array_equal(Q, Qr)


def test_fp8_code_book_grid_ties_and_tiny_values():
    vals = oracle.e4m3_decode(np.arange(1, 0x7F, dtype=np.uint8))
    row = np.zeros(512, np.float64)
    row[:126] = vals
    row[126:252] = -vals
    # midpoints between neighbouring codes (BF16-exact: at most 5 significant bits) and values below the
    # smallest subnormal step, next to a 448 that makes the reciprocal exactly 1
    d = oracle.e4m3_decode(np.arange(0, 0x7F, dtype=np.uint8))
    mids = (d[:-1] + d[1:]) / 2
    row2 = np.zeros(512, np.float64)
    row2[0] = 448.0
    row2[1:127] = mids
    row2[127:130] = [2.0 ** -10, 2.0 ** -11, 3 * 2.0 ** -11]
    A = inputs.f32_to_bf16_bits(np.stack([row, row2]).astype(np.float32))
    assert np.array_equal(inputs.bf16_bits_to_f32(A).astype(np.float64), np.stack([row, row2]))
    Q, S = gpu_quantize(A)
    Qr, Sr = oracle.quantize_rows_fp8(A)
    assert np.array_equal(Q, Qr) and np.array_equal(S, Sr)
    assert np.array_equal(Q[0, :126], np.arange(1, 0x7F)) and S[0] == 1.0 and S[1] == 1.0
    assert np.array_equal(Q[1, 1:127], np.where(np.arange(126) % 2 == 0, np.arange(126), np.arange(126) + 1))


def test_fp8_gate_up_and_rmsnorm_code_books():
    I, K = 520, 1040
    Wg = inputs.normal_bf16(710, "W", (I, K), 0.03)
    Wu = inputs.normal_bf16(711, "W", (I, K), 0.05)
    Qg, Qu = (torch.zeros((I, K), dtype=torch.uint8, device="cuda").view(F8) for _ in range(2))
    Sg, Su = (torch.zeros((I,), dtype=torch.float32, device="cuda") for _ in range(2))
    kx.kx_quantize_gate_up_fp8(kt.to_dev(Wg), kt.to_dev(Wu), Qg, Sg, Qu, Su)
    for Q, S, W in ((Qg, Sg, Wg), (Qu, Su, Wu)):
        Qr, Sr = oracle.quantize_rows_fp8(W)
        assert np.array_equal(host8(Q), Qr) and np.array_equal(S.cpu().numpy(), Sr)
    for (M, N) in [(130, 4096), (1000, 5120), (9, 32768), (7, 3072), (3, 8192), (9, 7168), (9000, 256)]:
        H = inputs.normal_bf16(720 + N, "R", (M, N), 1.3)
        g = inputs.normal_bf16(720 + N, "bias", (N,), 1.0)
        Z = kt.nan_filled(M, N)
        kx.kx_rmsnorm(kt.to_dev(H), kt.to_dev(g), 1e-6, Z)
        Q = torch.zeros((M, N), dtype=torch.uint8, device="cuda").view(F8)
        S = torch.zeros((M,), dtype=torch.float32, device="cuda")
        kx.kx_rmsnorm_quantize_fp8(kt.to_dev(H), kt.to_dev(g), 1e-6, Q, S)
        Qr, Sr = oracle.quantize_rows_fp8(kt.from_dev(Z))       # the device's own BF16 RMSNorm output
        assert np.array_equal(host8(Q), Qr) and np.array_equal(S.cpu().numpy(), Sr)


# ------------------------------------------------------------------ FP8 GEMMs
SMALL = np.array([0x00, 0x30, 0x38, 0x40, 0x48, 0xB0, 0xB8, 0xC0, 0xC8], dtype=np.uint8)   # 0, +-0.5, +-1, +-2, +-4


def small_codes(seed, shape):
    return SMALL[np.random.default_rng(seed).integers(0, len(SMALL), size=shape)]


def data_codes(seed, name, shape, std):
    """Codes and scales of normally distributed data, as the code book produces them."""
    return oracle.quantize_rows_fp8(inputs.normal_bf16(seed, name, shape, std))


def run_proj(Xq, sx, Wq, sw, b=None, R=None, inplace=False):
    M, N = Xq.shape[0], Wq.shape[0]
    if inplace:
        Y = kt.to_dev(R)
        Rd = Y
    else:
        Y = kt.nan_filled(M, N)
        Rd = kt.to_dev(R)
    kx.kx_outproj_residual_fp8(dev8(Xq), dev(sx), dev8(Wq), dev(sw), kt.to_dev(b), Rd, Y)
    status_ok()
    return kt.from_dev(Y)


def pow2(seed, n, lo=-10, hi=-4):
    return (2.0 ** np.random.default_rng(seed).integers(lo, hi + 1, size=n)).astype(np.float32)


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (300, 520, 272), (640, 1024, 512), (1000, 776, 1040), (7, 64, 16),
                                   (2048, 4096, 256), (2500, 3080, 400), (384, 512, 14336)])
def test_fp8_projection_exact_on_small_values(M, N, K):
    """Operand values in {0, +-0.5, +-1, +-2, +-4}: every product is a multiple of 1/4 of size at most 16 and
    every partial sum an exactly representable multiple of 1/4 (|sum| <= 16 K < 2^18), so any accumulation
    order and any internal alignment give the exact sum; power-of-two scales, single BF16 rounding."""
    Xq, Wq = small_codes(800 + M, (M, K)), small_codes(801 + N, (N, K))
    sx, sw = pow2(802, M), pow2(803, N)
    ok, msg = kt.gate_exact(run_proj(Xq, sx, Wq, sw), oracle.outproj_fp8(Xq, sx, Wq, sw))
    assert ok, msg


def test_fp8_projection_exact_with_small_integer_epilogue():
    M, N, K = 600, 776, 96
    vals = np.array([0x00, 0x38, 0xB8], dtype=np.uint8)                     # 0, +-1
    rng = np.random.default_rng(810)
    Xq, Wq = vals[rng.integers(0, 3, (M, K))], vals[rng.integers(0, 3, (N, K))]
    one_m, one_n = np.ones(M, np.float32), np.ones(N, np.float32)
    b = inputs.small_int_bf16(812, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(812, "R", (M, N), -8, 8)
    y = run_proj(Xq, one_m, Wq, one_n, b, R)
    ok, msg = kt.gate_exact(y, oracle.outproj_fp8(Xq, one_m, Wq, one_n, b, R))
    assert ok, msg
    assert np.array_equal(run_proj(Xq, one_m, Wq, one_n, b, R.copy(), inplace=True), y)


@pytest.mark.parametrize("M,N,K", [(300, 520, 272), (1000, 776, 1040), (2500, 3080, 4096)])
def test_fp8_projection_realistic_codes(M, N, K):
    """Codes and scales of normal data, bias and residual.  The hardware accumulates FP8 products in FP32;
    the gates are those of the BF16 path (formal tolerance, relative Frobenius error, determinism)."""
    Xq, sx = data_codes(820 + M, "X", (M, K), 1.0)
    Wq, sw = data_codes(821, "W", (N, K), 1.0 / np.sqrt(K))
    b = inputs.normal_bf16(824, "bias", (N,), 0.1)
    R = inputs.normal_bf16(824, "R", (M, N), 1.0)
    y = run_proj(Xq, sx, Wq, sw, b, R)
    ref = oracle.outproj_fp8(Xq, sx, Wq, sw, b, R)
    ok, msg = kt.gate_a(y, ref)
    assert ok, msg
    assert kt.rel_fro(y, ref) <= 2.0 ** -8
    y0 = run_proj(Xq, sx, Wq, sw)
    ref0 = oracle.outproj_fp8(Xq, sx, Wq, sw)
    assert kt.rel_fro(y0, ref0) <= 2.0 ** -8                                 # the GEMM term on its own
    assert np.array_equal(run_proj(Xq, sx, Wq, sw, b, R), y)


def run_swiglu(Xq, sx, Wgq, sg, Wuq, su):
    M, I = Xq.shape[0], Wgq.shape[0]
    Z = kt.nan_filled(M, I)
    kx.kx_gate_up_swiglu_fp8(dev8(Xq), dev(sx), dev8(Wgq), dev(sg), dev8(Wuq), dev(su), Z)
    status_ok()
    return kt.from_dev(Z)


def check_swiglu(z_bits, ref):
    ok, msg = kt.gate_a(z_bits, ref)
    assert ok, msg
    assert kt.rel_fro(z_bits, ref) <= 2.0 ** -8
    z = oracle.widen_bf16(z_bits)
    assert (np.abs(z - ref) <= 2.0 ** -7 * np.abs(ref) + 2e-3).all()


@pytest.mark.parametrize("M,I,K", [(128, 128, 128), (300, 520, 272), (640, 1024, 512), (7, 776, 1104),
                                   (2048, 4096, 512), (2500, 3080, 272)])
def test_fp8_swiglu_matches_oracle(M, I, K):
    Xq, sx = data_codes(830 + M, "X", (M, K), 1.0)
    Wgq, sg = data_codes(831, "W", (I, K), 1.0 / np.sqrt(K))
    Wuq, su = data_codes(832, "W", (I, K), 1.0 / np.sqrt(K))
    check_swiglu(run_swiglu(Xq, sx, Wgq, sg, Wuq, su), oracle.swiglu_fp8(Xq, sx, Wgq, sg, Wuq, su))


def test_fp8_swiglu_exact_pins_and_pairing():
    M, I, K = 384, 520, 320
    Xq, sx = data_codes(840, "X", (M, K), 1.0)
    Wgq, sg = data_codes(841, "W", (I, K), 1.0 / np.sqrt(K))
    Wuq, su = data_codes(842, "W", (I, K), 1.0 / np.sqrt(K))
    z = run_swiglu(Xq, sx, Wgq, sg, Wuq, su)
    zero = np.zeros_like(Wgq)
    assert not (run_swiglu(Xq, sx, zero, sg, Wuq, su) & 0x7FFF).any()
    assert not (run_swiglu(Xq, sx, Wgq, sg, zero, su) & 0x7FFF).any()
    want = inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(z))
    assert np.array_equal(run_swiglu(Xq, sx, Wgq, sg, Wuq, (2 * su).astype(np.float32)), want)
    assert np.array_equal(run_swiglu(Xq, sx, Wgq, sg, Wuq, su), z)
    # one-hot code rows (value 1) select single weights: fixes the gate/up pairing and the scale axes
    M2, K2 = 260, 448
    Xo = np.zeros((M2, K2), np.uint8)
    Xo[np.arange(M2), np.arange(M2) % K2] = 0x38
    Wg2, Wu2 = small_codes(843, (I, K2)), small_codes(844, (I, K2))
    s1 = np.ones(M2, np.float32)
    sg2, su2 = pow2(845, I, -2, 1), pow2(846, I, -3, 0)
    zz = oracle.widen_bf16(run_swiglu(Xo, s1, Wg2, sg2, Wu2, su2))
    g = oracle.e4m3_decode(Wg2)[:, np.arange(M2) % K2].T * sg2[None, :]
    u = oracle.e4m3_decode(Wu2)[:, np.arange(M2) % K2].T * su2[None, :]
    ref = g / (1.0 + np.exp(-g)) * u
    assert (np.abs(zz - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-6).all()


def test_fp8_edge_cases_and_errors():
    lib = kx.load()
    A = 0x100000
    Z = kt.nan_filled(5, 16)
    assert lib.kx_gate_up_swiglu_fp8(None, None, None, None, None, None, Z.data_ptr(), 5, 16, 0, None) == kx.KX_OK
    assert not kt.from_dev(Z).any()
    assert lib.kx_gate_up_swiglu_fp8(A, 2 * A, 3 * A, 4 * A, 5 * A, 6 * A, 7 * A, 5, 16, 24, None) == kx.KX_ERR_SHAPE
    assert lib.kx_outproj_residual_fp8(A, 2 * A, 3 * A, 4 * A, None, None, A, 5, 16, 16, None) == kx.KX_ERR_OVERLAP
    assert lib.kx_quantize_rows_fp8(A, 2 * A, 4 * A, 4, 24, None) == kx.KX_ERR_SHAPE
    assert lib.kx_quantize_rows_fp8(A, None, 4 * A, 4, 32, None) == kx.KX_ERR_NULL


def test_fp8_mlp_chain_full_size_sampled_rows():
    """RMSNorm + FP8 code book -> weights' code books in one launch -> FP8 gate/up + SwiGLU at the decoder
    layer's size (4096 tokens, hidden 4096, intermediate 14336), sampled rows of every stage against the
    oracle applied to that stage's device-produced input."""
    M, Hd, I = 4096, 4096, 14336
    H = inputs.normal_bf16(850, "R", (M, Hd), 1.0)
    g = inputs.normal_bf16(850, "bias", (Hd,), 1.0)
    Wg = inputs.normal_bf16(851, "W", (I, Hd), 1.0 / np.sqrt(Hd))
    Wu = inputs.normal_bf16(852, "W", (I, Hd), 1.0 / np.sqrt(Hd))
    Xq = torch.empty((M, Hd), dtype=torch.uint8, device="cuda").view(F8)
    Qg, Qu = (torch.empty((I, Hd), dtype=torch.uint8, device="cuda").view(F8) for _ in range(2))
    sx = torch.empty((M,), dtype=torch.float32, device="cuda")
    Sg, Su = (torch.empty((I,), dtype=torch.float32, device="cuda") for _ in range(2))
    Z = kt.nan_filled(M, I)
    kx.kx_rmsnorm_quantize_fp8(kt.to_dev(H), kt.to_dev(g), 1e-6, Xq, sx)
    kx.kx_quantize_gate_up_fp8(kt.to_dev(Wg), kt.to_dev(Wu), Qg, Sg, Qu, Su)
    kx.kx_gate_up_swiglu_fp8(Xq, sx, Qg, Sg, Qu, Su, Z)
    status_ok()
    xq, sxh = host8(Xq), sx.cpu().numpy()
    qg, qu, sgh, suh = host8(Qg), host8(Qu), Sg.cpu().numpy(), Su.cpu().numpy()
    Qr, Sr = oracle.quantize_rows_fp8(Wu)
    assert np.array_equal(qu, Qr) and np.array_equal(suh, Sr)
    rows = inputs.sampled_rows(M)[::4]
    z = kt.from_dev(Z)
    assert not np.isnan(oracle.widen_bf16(z)).any()
    check_swiglu(z[rows], oracle.swiglu_fp8(xq, sxh, qg, sgh, qu, suh, rows=rows))
    zn = oracle.round_bf16(oracle.rmsnorm(H, g, 1e-6, rows=rows[:8]))
    ref16 = oracle.swiglu(zn, Wg, Wu)
    z8 = oracle.widen_bf16(z[rows[:8]])
    assert np.sqrt(np.mean((z8 - ref16) ** 2)) / np.sqrt(np.mean(ref16 ** 2)) < 0.08


@pytest.mark.parametrize("M,N,K", [(4096, 4096, 4096), (16384, 4096, 14336)])
def test_fp8_projection_full_sizes_sampled_rows(M, N, K):
    """The two projection shapes bench.py times for FP8, in that launch configuration: exact on the
    small-value code set, then realistic codes with a residual within the gates (sampled rows)."""
    Xq, Wq = small_codes(860, (M, K)), small_codes(861, (N, K))
    sx, sw = pow2(862, M), pow2(863, N)
    rows = inputs.sampled_rows(M)[::8]
    Y = kt.nan_filled(M, N)
    kx.kx_outproj_residual_fp8(dev8(Xq), dev(sx), dev8(Wq), dev(sw), None, None, Y)
    status_ok()
    y = kt.from_dev(Y)
    assert not np.isnan(oracle.widen_bf16(y)).any()
    ok, msg = kt.gate_exact(y[rows], oracle.outproj_fp8(Xq, sx, Wq, sw, rows=rows))
    assert ok, msg
    Xq2, sx2 = data_codes(864, "X", (M, K), 1.0)
    Wq2, sw2 = data_codes(865, "W", (N, K), 1.0 / np.sqrt(K))
    R = inputs.normal_bf16(866, "R", (M, N), 1.0)
    kx.kx_outproj_residual_fp8(dev8(Xq2), dev(sx2), dev8(Wq2), dev(sw2), None, kt.to_dev(R), Y)
    status_ok()
    y = kt.from_dev(Y)
    ref = oracle.outproj_fp8(Xq2, sx2, Wq2, sw2, None, R, rows=rows)
    ok, msg = kt.gate_a(y[rows], ref)
    assert ok, msg
    assert kt.rel_fro(y[rows], ref) <= 2.0 ** -8
