"""INT8 branch (row code books, RMSNorm + quantisation, INT8 gate/up + SwiGLU, INT8 projection
with residual): the CUDA kernels, through the C ABI, against the CPU oracle.  Codes and scales
are compared bit for bit; the integer GEMM bit for bit wherever the dequantised value has a
single rounding; everything else with the tolerance gates of the BF16 path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def status_ok():
    code, detail = kx.kx_last_device_status()
    assert code == kx.KX_OK, (code, detail)


# ------------------------------------------------------------------ code books
def gpu_quantize(A):
    rows, cols = A.shape
    Q = torch.full((rows, cols), 77, dtype=torch.int8, device="cuda")
    S = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda")
    kx.kx_quantize_rows_int8(kt.to_dev(A), Q, S)
    return Q.cpu().numpy(), S.cpu().numpy()


@pytest.mark.parametrize("rows,cols", [(1, 16), (5, 48), (300, 2064), (129, 4096), (40, 8192), (3, 32768), (700, 1024), (7, 3072), (5, 2560), (9, 7168), (5, 6144), (9000, 256)])
def test_quantize_rows_bit_exact(rows, cols):
    A = inputs.normal_bf16(500 + cols, "X", (rows, cols), 2.5)
    if rows > 2:
        A[1] = 0                                   # a zero row: scale 1, codes 0
        A[2, : cols // 2] = 0
    Q, S = gpu_quantize(A)
    Qr, Sr = oracle.quantize_rows(A)
    assert np.array_equal(S.view(np.uint32), Sr.view(np.uint32))
    assert np.array_equal(Q, Qr)


def test_quantize_ties_and_grid():
    j = np.arange(-127, 128, dtype=np.float32)
    row = np.concatenate([j, np.zeros(1, np.float32)]) * np.float32(2.0 ** -6)
    ties = np.zeros(256, np.float32)
    ties[:11] = np.array([127.0, 0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, 62.5, 63.5, -63.5], np.float32) * 0.25
    A = inputs.f32_to_bf16_bits(np.stack([row, ties]))
    Q, S = gpu_quantize(A)
    assert np.array_equal(Q[0, :255], j.astype(np.int8)) and S[0] == np.float32(2.0 ** -6)
    assert np.array_equal(Q[1, :11], np.array([127, 0, 2, 2, 4, 0, -2, -2, 62, 64, -64], np.int8))
    Qr, Sr = oracle.quantize_rows(A)
    assert np.array_equal(Q, Qr) and np.array_equal(S, Sr)


def test_quantize_gate_and_up_in_one_launch():
    I, K = 520, 1040
    Wg = inputs.normal_bf16(510, "W", (I, K), 0.03)
    Wu = inputs.normal_bf16(511, "W", (I, K), 0.05)
    Qg = torch.zeros((I, K), dtype=torch.int8, device="cuda")
    Qu = torch.zeros((I, K), dtype=torch.int8, device="cuda")
    Sg = torch.zeros((I,), dtype=torch.float32, device="cuda")
    Su = torch.zeros((I,), dtype=torch.float32, device="cuda")
    kx.kx_quantize_gate_up_int8(kt.to_dev(Wg), kt.to_dev(Wu), Qg, Sg, Qu, Su)
    for Q, S, W in ((Qg, Sg, Wg), (Qu, Su, Wu)):
        Qr, Sr = oracle.quantize_rows(W)
        assert np.array_equal(Q.cpu().numpy(), Qr) and np.array_equal(S.cpu().numpy(), Sr)


@pytest.mark.parametrize("M,N", [(3, 272), (130, 4096), (9, 32768), (1000, 5120), (2500, 2048), (7, 3072), (3, 8192), (5, 6144), (9, 7168), (5, 2560), (9000, 256)])
def test_rmsnorm_quantize(M, N):
    """The fused kernel quantises exactly the BF16 values kx_rmsnorm writes: the code book of
    that (device-computed) z, taken by the oracle, must be reproduced bit for bit; z itself is
    checked against the oracle's RMSNorm in its own test file.  End to end against the oracle
    chain the dequantised value stays within half a code step plus one BF16 ulp of z."""
    eps = 1e-6
    H = inputs.normal_bf16(520 + N, "R", (M, N), 1.3)
    g = inputs.normal_bf16(520 + N, "bias", (N,), 1.0)
    Z = kt.nan_filled(M, N)
    kx.kx_rmsnorm(kt.to_dev(H), kt.to_dev(g), eps, Z)
    z_bits = kt.from_dev(Z)
    Q = torch.full((M, N), 77, dtype=torch.int8, device="cuda")
    S = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
    kx.kx_rmsnorm_quantize_int8(kt.to_dev(H), kt.to_dev(g), eps, Q, S)
    Qr, Sr = oracle.quantize_rows(z_bits)
    q, s = Q.cpu().numpy(), S.cpu().numpy()
    assert np.array_equal(s, Sr) and np.array_equal(q, Qr)
    zref = oracle.rmsnorm(H, g, eps)
    err = np.abs(q.astype(np.float64) * s[:, None].astype(np.float64) - zref)
    assert (err <= 0.5 * s[:, None] * (1 + 1e-5) + 2.0 ** -8 * np.abs(zref)).all()


def test_quantize_errors():
    A = 0x100000
    lib = kx.load()
    assert lib.kx_quantize_rows_int8(A, 2 * A, 4 * A, 4, 24, None) == kx.KX_ERR_SHAPE      # cols % 16
    assert lib.kx_quantize_rows_int8(A, 2 * A, 4 * A, 4, 65536, None) == kx.KX_ERR_SHAPE   # too wide
    assert lib.kx_quantize_rows_int8(A, None, 4 * A, 4, 32, None) == kx.KX_ERR_NULL
    assert lib.kx_quantize_rows_int8(A, A + 64, 4 * A, 4, 32, None) == kx.KX_ERR_OVERLAP
    assert lib.kx_quantize_rows_int8(A, 2 * A + 4, 4 * A, 4, 32, None) == kx.KX_ERR_ALIGN
    assert lib.kx_quantize_rows_int8(A, 2 * A, 4 * A, 0, 32, None) == kx.KX_OK
    assert lib.kx_rmsnorm_quantize_int8(A, None, 1e-6, 2 * A, 4 * A, 4, 32, None) == kx.KX_ERR_NULL
    assert lib.kx_rmsnorm_quantize_int8(A, 8 * A, -1.0, 2 * A, 4 * A, 4, 32, None) == kx.KX_ERR_SHAPE


# ------------------------------------------------------------------ INT8 GEMMs
def codes(seed, shape, lo=-127, hi=127):
    return np.random.default_rng(seed).integers(lo, hi + 1, size=shape, dtype=np.int8)


def pow2(seed, n, lo=-12, hi=-6):
    return (2.0 ** np.random.default_rng(seed).integers(lo, hi + 1, size=n)).astype(np.float32)


def scales(seed, n, mid):
    return (mid * np.exp(np.random.default_rng(seed).normal(0, 0.3, size=n))).astype(np.float32)


def run_proj(Xq, sx, Wq, sw, b=None, R=None, inplace=False):
    M, N = Xq.shape[0], Wq.shape[0]
    if inplace:
        Y = kt.to_dev(R)
        Rd = Y
    else:
        Y = kt.nan_filled(M, N)
        Rd = kt.to_dev(R)
    kx.kx_outproj_residual_int8(dev(Xq), dev(sx), dev(Wq), dev(sw), kt.to_dev(b), Rd, Y)
    status_ok()
    return kt.from_dev(Y)


# shapes cover single-CTA tiles of every width, CTA pairs (enough 256-row tiles), ragged M / N / K
SHAPES = [(128, 256, 128), (300, 520, 272), (640, 1024, 512), (1000, 776, 1040), (7, 64, 16),
          (2048, 4096, 256), (2500, 3080, 400)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_int8_projection_exact_integer_sum(M, N, K):
    """Full-range codes, K <= 1040: |sum| < 2^24, so its FP32 image is exact; power-of-two scales
    multiply exactly; with no bias / residual the only rounding is the one to BF16 -> the output
    equals the once-rounded exact value bit for bit, for every accumulation the tensor core did."""
    Xq, Wq = codes(600 + M, (M, K)), codes(601 + N, (N, K))
    sx, sw = pow2(602, M), pow2(603, N)
    y = run_proj(Xq, sx, Wq, sw)
    ok, msg = kt.gate_exact(y, oracle.outproj_int8(Xq, sx, Wq, sw))
    assert ok, msg


def test_int8_projection_exact_with_small_integer_epilogue():
    """Ternary codes, unit scales, small-integer bias and residual: every value is an integer below
    2^8, so the whole epilogue is exact and in-place operation gives the same bits."""
    M, N, K = 600, 776, 96
    Xq, Wq = codes(610, (M, K), -1, 1), codes(611, (N, K), -1, 1)
    one_m, one_n = np.ones(M, np.float32), np.ones(N, np.float32)
    b = inputs.small_int_bf16(612, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(612, "R", (M, N), -8, 8)
    y = run_proj(Xq, one_m, Wq, one_n, b, R)
    ok, msg = kt.gate_exact(y, oracle.outproj_int8(Xq, one_m, Wq, one_n, b, R))
    assert ok, msg
    assert np.array_equal(run_proj(Xq, one_m, Wq, one_n, b, R.copy(), inplace=True), y)


def test_int8_projection_long_reduction_exact():
    """K = 14336 (the down projection's reduction length): codes in -15..15 keep |sum| < 2^24."""
    M, N, K = 384, 512, 14336
    Xq, Wq = codes(620, (M, K), -15, 15), codes(621, (N, K), -15, 15)
    sx, sw = pow2(622, M), pow2(623, N)
    ok, msg = kt.gate_exact(run_proj(Xq, sx, Wq, sw), oracle.outproj_int8(Xq, sx, Wq, sw))
    assert ok, msg


@pytest.mark.parametrize("M,N,K", [(300, 520, 272), (1000, 776, 1040), (2500, 3080, 4096)])
def test_int8_projection_general_scales(M, N, K):
    """Arbitrary FP32 scales, bias and residual: formal tolerance, and at most one BF16 ulp."""
    Xq, Wq = codes(630 + M, (M, K)), codes(631, (N, K))
    sx, sw = scales(632, M, 0.02), scales(633, N, 4e-4 / np.sqrt(K / 1024))
    b = inputs.normal_bf16(634, "bias", (N,), 0.1)
    R = inputs.normal_bf16(634, "R", (M, N), 1.0)
    y = run_proj(Xq, sx, Wq, sw, b, R)
    ref = oracle.outproj_int8(Xq, sx, Wq, sw, b, R)
    ok, msg = kt.gate_a(y, ref)
    assert ok, msg
    err = np.abs(oracle.widen_bf16(y) - ref)
    assert (err <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -8 * (np.abs(oracle.widen_bf16(R)) + 0.5)).all()
    assert float((oracle.round_bf16(ref) != y).mean()) <= 0.01
    assert np.array_equal(run_proj(Xq, sx, Wq, sw, b, R), y)       # deterministic


def test_int8_projection_scale_axes_and_selectors():
    """One-hot code rows pick single weight codes: y[m,n] = 127 * Wq[n, m mod K] * sx[m] * sw[n];
    a transposed scale vector or operand would be off by O(1)."""
    M, N, K = 300, 264, 144
    Xq = np.zeros((M, K), np.int8)
    Xq[np.arange(M), np.arange(M) % K] = 127
    Wq = codes(640, (N, K))
    sx, sw = pow2(641, M), pow2(642, N, -3, 3)
    y = oracle.widen_bf16(run_proj(Xq, sx, Wq, sw))
    want = 127.0 * Wq[:, np.arange(M) % K].T.astype(np.float64) * sx[:, None] * sw[None, :]
    assert np.array_equal(y, oracle.widen_bf16(oracle.round_bf16(want)))


def run_swiglu(Xq, sx, Wgq, sg, Wuq, su):
    M, I = Xq.shape[0], Wgq.shape[0]
    Z = kt.nan_filled(M, I)
    kx.kx_gate_up_swiglu_int8(dev(Xq), dev(sx), dev(Wgq), dev(sg), dev(Wuq), dev(su), Z)
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
def test_int8_swiglu_matches_oracle(M, I, K):
    Xq, Wgq, Wuq = codes(650 + M, (M, K)), codes(651, (I, K)), codes(652, (I, K))
    amp = 1.0 / (73.0 * 73.0 * np.sqrt(K))        # pre-activations of order one
    sx, sg, su = scales(653, M, 1.0), scales(654, I, amp), scales(655, I, amp)
    ref, ga, ua = oracle.swiglu_int8(Xq, sx, Wgq, sg, Wuq, su, want_acc=True)
    check_swiglu(run_swiglu(Xq, sx, Wgq, sg, Wuq, su), ref)
    assert 0.3 < np.abs(ga * sx[:, None] * sg[None, :]).std() < 3.0


def test_int8_swiglu_exact_pins():
    M, I, K = 384, 520, 320
    Xq, Wgq, Wuq = codes(660, (M, K)), codes(661, (I, K)), codes(662, (I, K))
    amp = 1.0 / (73.0 * 73.0 * np.sqrt(K))
    sx, sg, su = scales(663, M, 1.0), scales(664, I, amp), scales(665, I, amp)
    z = run_swiglu(Xq, sx, Wgq, sg, Wuq, su)
    zero = np.zeros_like(Wgq)
    assert not (run_swiglu(Xq, sx, zero, sg, Wuq, su) & 0x7FFF).any()        # silu(0) * u = 0
    assert not (run_swiglu(Xq, sx, Wgq, sg, zero, su) & 0x7FFF).any()        # silu(g) * 0 = 0
    want = inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(z))
    assert np.array_equal(run_swiglu(Xq, sx, Wgq, sg, Wuq, (2 * su).astype(np.float32)), want)   # linear in su
    assert np.array_equal(run_swiglu(Xq, sx, Wgq, sg, Wuq, su), z)                              # deterministic


def test_int8_swiglu_selectors_fix_the_gate_up_pairing():
    M, I, K = 260, 392, 448
    Xq = np.zeros((M, K), np.int8)
    Xq[np.arange(M), np.arange(M) % K] = 1
    Wgq, Wuq = codes(670, (I, K)), codes(671, (I, K))
    sx = np.ones(M, np.float32)
    sg, su = np.full(I, 2.0 ** -5, np.float32), np.full(I, 2.0 ** -6, np.float32)
    z = oracle.widen_bf16(run_swiglu(Xq, sx, Wgq, sg, Wuq, su))
    g = Wgq[:, np.arange(M) % K].T.astype(np.float64) * 2.0 ** -5
    u = Wuq[:, np.arange(M) % K].T.astype(np.float64) * 2.0 ** -6
    ref = g / (1.0 + np.exp(-g)) * u
    assert (np.abs(z - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-6).all()


def test_int8_edge_cases_and_errors():
    M, I, K = 5, 16, 16
    Xq, Wgq, Wuq = codes(680, (M, K)), codes(681, (I, K)), codes(682, (I, K))
    sx, sg, su = scales(683, M, 1.0), scales(684, I, 1e-3), scales(685, I, 1e-3)
    check_swiglu(run_swiglu(Xq, sx, Wgq, sg, Wuq, su), oracle.swiglu_int8(Xq, sx, Wgq, sg, Wuq, su))
    lib = kx.load()
    A = 0x100000
    Z = kt.nan_filled(5, 16)
    assert lib.kx_gate_up_swiglu_int8(None, None, None, None, None, None, Z.data_ptr(), 5, 16, 0, None) == kx.KX_OK
    assert not kt.from_dev(Z).any()                                          # empty sums
    R = inputs.small_int_bf16(686, "R", (5, 16), -8, 8)
    Y = kt.nan_filled(5, 16)
    assert lib.kx_outproj_residual_int8(None, None, None, None, None, kt.to_dev(R).data_ptr(), Y.data_ptr(), 5, 16, 0,
                                        None) == kx.KX_OK
    torch.cuda.synchronize()
    assert np.array_equal(kt.from_dev(Y), R)
    args = lambda K_, I_=16: (A, 2 * A, 3 * A, 4 * A, 5 * A, 6 * A, 7 * A, 5, I_, K_, None)
    assert lib.kx_gate_up_swiglu_int8(*args(24)) == kx.KX_ERR_SHAPE           # K % 16
    assert lib.kx_gate_up_swiglu_int8(*args(16, 12)) == kx.KX_ERR_SHAPE       # I % 8
    assert lib.kx_gate_up_swiglu_int8(A, None, 3 * A, 4 * A, 5 * A, 6 * A, 7 * A, 5, 16, 16, None) == kx.KX_ERR_NULL
    assert lib.kx_gate_up_swiglu_int8(A, 2 * A, 3 * A, 4 * A + 4, 5 * A, 6 * A, 7 * A, 5, 16, 16, None) == kx.KX_ERR_ALIGN
    assert lib.kx_outproj_residual_int8(A, 2 * A, 3 * A, 4 * A, None, None, A, 5, 16, 16, None) == kx.KX_ERR_OVERLAP


def test_int8_mlp_chain_full_size_sampled_rows():
    """The INT8 branch end to end at the decoder layer's size: h -> RMSNorm + quantise -> INT8
    gate/up + SwiGLU with weights quantised in one launch, M = 4096 tokens, hidden 4096,
    intermediate 14336.  Every stage is checked on sampled rows against the oracle applied to the
    device-produced input of that stage."""
    M, Hd, I = 4096, 4096, 14336
    H = inputs.normal_bf16(690, "R", (M, Hd), 1.0)
    g = inputs.normal_bf16(690, "bias", (Hd,), 1.0)
    Wg = inputs.normal_bf16(691, "W", (I, Hd), 1.0 / np.sqrt(Hd))
    Wu = inputs.normal_bf16(692, "W", (I, Hd), 1.0 / np.sqrt(Hd))
    Xq = torch.empty((M, Hd), dtype=torch.int8, device="cuda")
    sx = torch.empty((M,), dtype=torch.float32, device="cuda")
    Qg = torch.empty((I, Hd), dtype=torch.int8, device="cuda")
    Qu = torch.empty((I, Hd), dtype=torch.int8, device="cuda")
    Sg = torch.empty((I,), dtype=torch.float32, device="cuda")
    Su = torch.empty((I,), dtype=torch.float32, device="cuda")
    Z = kt.nan_filled(M, I)
    kx.kx_rmsnorm_quantize_int8(kt.to_dev(H), kt.to_dev(g), 1e-6, Xq, sx)
    kx.kx_quantize_gate_up_int8(kt.to_dev(Wg), kt.to_dev(Wu), Qg, Sg, Qu, Su)
    kx.kx_gate_up_swiglu_int8(Xq, sx, Qg, Sg, Qu, Su, Z)
    status_ok()
    xq, sxh = Xq.cpu().numpy(), sx.cpu().numpy()
    qg, qu, sgh, suh = Qg.cpu().numpy(), Qu.cpu().numpy(), Sg.cpu().numpy(), Su.cpu().numpy()
    Qr, Sr = oracle.quantize_rows(Wg)
    assert np.array_equal(qg, Qr) and np.array_equal(sgh, Sr)
    rows = inputs.sampled_rows(M)[::4]
    z = kt.from_dev(Z)
    assert not np.isnan(oracle.widen_bf16(z)).any()
    check_swiglu(z[rows], oracle.swiglu_int8(xq, sxh, qg, sgh, qu, suh, rows=rows))
    # and the quantised branch tracks the BF16 branch it replaces (code-book error, not a bug's O(1))
    zn = oracle.round_bf16(oracle.rmsnorm(H, g, 1e-6, rows=rows[:8]))
    ref16 = oracle.swiglu(zn, Wg, Wu)
    z8 = oracle.widen_bf16(z[rows[:8]])
    assert np.sqrt(np.mean((z8 - ref16) ** 2)) / np.sqrt(np.mean(ref16 ** 2)) < 0.05


@pytest.mark.parametrize("M,N,K", [(4096, 4096, 4096), (16384, 4096, 14336)])
def test_int8_projection_full_sizes_sampled_rows(M, N, K):
    """The two projection shapes bench.py times in its 8-bit section, in that launch configuration:
    codes in -15..15 keep every sum below 2^24, so with power-of-two scales and no bias / residual the
    sampled rows must be bit-exact; then general scales with a residual within the gates."""
    rng = np.random.default_rng(695)
    Xq = rng.integers(-15, 16, size=(M, K), dtype=np.int8)
    Wq = rng.integers(-15, 16, size=(N, K), dtype=np.int8)
    sx, sw = pow2(696, M), pow2(697, N)
    rows = inputs.sampled_rows(M)[::8]
    Xd, Wd = dev(Xq), dev(Wq)
    Y = kt.nan_filled(M, N)
    kx.kx_outproj_residual_int8(Xd, dev(sx), Wd, dev(sw), None, None, Y)
    status_ok()
    y = kt.from_dev(Y)
    assert not np.isnan(oracle.widen_bf16(y)).any()
    ok, msg = kt.gate_exact(y[rows], oracle.outproj_int8(Xq, sx, Wq, sw, rows=rows))
    assert ok, msg
    sx2, sw2 = scales(698, M, 0.05), scales(699, N, 0.02 / np.sqrt(K))
    R = inputs.normal_bf16(700, "R", (M, N), 1.0)
    kx.kx_outproj_residual_int8(Xd, dev(sx2), Wd, dev(sw2), None, kt.to_dev(R), Y)
    status_ok()
    y = kt.from_dev(Y)
    ref = oracle.outproj_int8(Xq, sx2, Wq, sw2, None, R, rows=rows)
    ok, msg = kt.gate_a(y[rows], ref)
    assert ok, msg
    assert float((oracle.round_bf16(ref) != y[rows]).mean()) <= 0.01
