"""Block-scaled FP8 branch: the code book (codes and chunked scale bytes) bit for bit, the
block-scaled projection bit for bit where every partial sum is exactly representable, the rest
within the tolerance gates of the BF16 path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu

F8 = torch.float8_e4m3fn


def dev8(codes):
    return torch.from_numpy(np.ascontiguousarray(codes)).cuda().view(F8)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host8(t):
    return t.view(torch.uint8).cpu().numpy()


def status_ok():
    code, detail = kx.kx_last_device_status()
    assert code == kx.KX_OK, (code, detail)


def chunked(E, cols):
    """Row-major scale bytes [rows, cols / 32] -> the library's chunked array (index arithmetic only;
    padding = 127)."""
    rows, nb = E.shape
    rc, kc = (rows + 127) // 128, (cols + 127) // 128
    out = np.full((rc, kc, 32, 4, 4), 127, dtype=np.uint8)           # [row chunk][k chunk][r % 32][r % 128 / 32][j % 4]
    r = np.arange(rows)[:, None]
    j = np.arange(nb)[None, :]
    out[r // 128, j // 4, r % 32, (r % 128) // 32, j % 4] = E
    return out.reshape(-1)


# ------------------------------------------------------------------ code book
def gpu_quantize(A):
    rows, cols = A.shape
    Q = torch.full((rows, cols), 0x55, dtype=torch.uint8, device="cuda").view(F8)
    SF = torch.full((kx.kx_mx_scale_bytes(rows, cols),), 0xEE, dtype=torch.uint8, device="cuda")
    kx.kx_quantize_rows_mxfp8(kt.to_dev(A), Q, SF)
    return host8(Q), SF.cpu().numpy()


def test_scale_bytes():
    assert kx.kx_mx_scale_bytes(1, 32) == 512 and kx.kx_mx_scale_bytes(128, 128) == 512
    assert kx.kx_mx_scale_bytes(129, 160) == 4 * 512 and kx.kx_mx_scale_bytes(0, 64) == 0
    assert kx.kx_mx_scale_bytes(-1, 64) < 0


@pytest.mark.parametrize("rows,cols", [(1, 32), (5, 96), (300, 2080), (129, 4096), (3, 32768), (700, 1024), (128, 128), (7, 3072), (5, 2560), (9, 7168), (5, 6144), (9000, 256)])
def test_mx_code_book_bit_exact(rows, cols):
    A = inputs.normal_bf16(900 + cols, "X", (rows, cols), 2.5)
    f = inputs.bf16_bits_to_f32(A)
    # blocks of very different magnitude in one row, a zero block, a zero row
    f[0, :32] *= 2.0 ** -40
    if cols >= 96:
        f[0, 32:64] *= 2.0 ** 30
        f[0, 64:96] = 0
    if rows > 2:
        f[1] = 0
    A = inputs.f32_to_bf16_bits(f)
    Q, SF = gpu_quantize(A)
    Qr, Er = oracle.quantize_rows_mx(A)
    assert np.array_equal(Q, Qr)
    assert np.array_equal(SF, chunked(Er, cols))


@pytest.mark.parametrize("M,N", [(130, 4096), (1000, 5120), (9, 32768), (300, 1056), (5, 32), (7, 3072), (3, 8192), (5, 6144), (9, 7168), (5, 2560), (9000, 256)])
def test_mx_rmsnorm_code_book(M, N):
    """Fused RMSNorm + code book = code book of the device's own BF16 RMSNorm output, bit for bit."""
    H = inputs.normal_bf16(950 + N, "R", (M, N), 1.3)
    g = inputs.normal_bf16(950 + N, "bias", (N,), 1.0)
    Z = kt.nan_filled(M, N)
    kx.kx_rmsnorm(kt.to_dev(H), kt.to_dev(g), 1e-6, Z)
    Q = torch.full((M, N), 0x55, dtype=torch.uint8, device="cuda").view(F8)
    SF = torch.full((kx.kx_mx_scale_bytes(M, N),), 0xEE, dtype=torch.uint8, device="cuda")
    kx.kx_rmsnorm_quantize_mxfp8(kt.to_dev(H), kt.to_dev(g), 1e-6, Q, SF)
    Qr, Er = oracle.quantize_rows_mx(kt.from_dev(Z))
    assert np.array_equal(host8(Q), Qr) and np.array_equal(SF.cpu().numpy(), chunked(Er, N))
    # and the RMSNorm itself is the oracle's within BF16 rounding (its own parity is tested elsewhere)
    ref = oracle.rmsnorm(H, g, 1e-6)
    assert kt.rel_fro(kt.from_dev(Z), ref) <= 2.0 ** -8


def test_mx_code_book_grid_and_saturation():
    vals = oracle.e4m3_decode(np.arange(0x5F, 0x7F, dtype=np.uint8))
    d = oracle.e4m3_decode(np.arange(0x40, 0x7F, dtype=np.uint8))
    mids = ((d[:-1] + d[1:]) / 2)[:31]
    row0 = np.concatenate([vals, -vals * 2.0 ** -9, np.r_[448.0, mids], np.r_[1.96875, 1.875, 1.75, np.zeros(29)]])
    A = inputs.f32_to_bf16_bits(row0.reshape(1, 128).astype(np.float32))
    assert np.array_equal(inputs.bf16_bits_to_f32(A).astype(np.float64), row0.reshape(1, 128))
    Q, SF = gpu_quantize(A)
    Qr, Er = oracle.quantize_rows_mx(A)
    assert np.array_equal(Q, Qr) and np.array_equal(SF, chunked(Er, 128))
    assert np.array_equal(Q[0, :32], np.arange(0x5F, 0x7F)) and Er[0].tolist() == [127, 118, 127, 119]
    assert Q[0, 96:99].tolist() == [0x7E, 0x7E, 0x7E]


# ------------------------------------------------------------------ projection
SMALL = np.array([0x00, 0x30, 0x38, 0x40, 0x48, 0xB0, 0xB8, 0xC0, 0xC8], dtype=np.uint8)   # 0, +-0.5, +-1, +-2, +-4


def small_codes(seed, shape):
    return SMALL[np.random.default_rng(seed).integers(0, len(SMALL), size=shape)]


# (tile columns, CTAs per tile, ring stages: 0 = default variant)
VARIANTS = [(128, 1, 0), (192, 1, 0), (128, 2, 0), (192, 2, 0), (256, 1, 0)]


def run_proj(Xq, ex, Wq, ew, b=None, R=None, inplace=False, variant=None):
    (M, K), N = Xq.shape, Wq.shape[0]
    ov = None if variant is None else kx.make_override(block_n=variant[0], cta_pair=variant[1], stages=variant[2])
    if inplace:
        Y = kt.to_dev(R)
        Rd = Y
    else:
        Y = kt.nan_filled(M, N)
        Rd = kt.to_dev(R)
    kx.kx_outproj_residual_mxfp8(dev8(Xq), dev(chunked(ex, K)), dev8(Wq), dev(chunked(ew, K)), kt.to_dev(b), Rd, Y,
                                 override=ov)
    status_ok()
    return kt.from_dev(Y)


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (128, 256, 256), (300, 520, 288), (640, 1024, 512), (1000, 776, 1056),
                                   (7, 64, 32), (2048, 4096, 256), (2500, 3080, 416), (384, 512, 8192),
                                   (130, 192, 160), (260, 960, 384), (4096, 4096 + 192, 128)])
def test_mx_projection_exact_on_small_values(M, N, K):
    """Element values in {0, +-0.5, +-1, +-2, +-4}, block scales in {1/2, 1, 2} (A) and {1/4, 1/2, 1} (B),
    drawn independently per (row, block): every product is a multiple of 2^-5 of size at most 32 and every
    partial sum is exactly representable (|sum| <= 32 K <= 2^18), so any accumulation order gives the exact
    sum - and a scale read from the wrong row, block or byte changes it."""
    rng = np.random.default_rng(900 + M + N + K)
    nb = K // 32
    Xq, Wq = small_codes(901 + M, (M, K)), small_codes(902 + N, (N, K))
    ex = rng.integers(126, 129, size=(M, nb), dtype=np.uint8)
    ew = rng.integers(125, 128, size=(N, nb), dtype=np.uint8)
    ok, msg = kt.gate_exact(run_proj(Xq, ex, Wq, ew), oracle.outproj_mx(Xq, ex, Wq, ew))
    assert ok, msg


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (300, 520, 288), (1000, 776, 1056), (7, 64, 32), (260, 960, 384),
                                   (2500, 3080, 416), (4096, 4096 + 192, 128)])
def test_mx_projection_every_tile_shape(variant, M, N, K):
    """The same exact-sum construction forced through each tile shape (single CTA / CTA pair, 128 / 192
    columns; with 192 columns every second tile starts in the middle of a scale chunk), with bias and R."""
    rng = np.random.default_rng(940 + M + N + K)
    nb = K // 32
    Xq, Wq = small_codes(941 + M, (M, K)), small_codes(942 + N, (N, K))
    ex = rng.integers(126, 129, size=(M, nb), dtype=np.uint8)
    ew = rng.integers(125, 128, size=(N, nb), dtype=np.uint8)
    b = inputs.small_int_bf16(943, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(943, "R", (M, N), -8, 8)
    ok, msg = kt.gate_exact(run_proj(Xq, ex, Wq, ew, b, R, variant=variant), oracle.outproj_mx(Xq, ex, Wq, ew, b, R))
    assert ok, msg


@pytest.mark.parametrize("chunk", range(4))
def test_mx_random_shapes_and_tile_shapes_are_exact(chunk):
    """Seeded random (M, N, K, tile shape, bias / residual / in place) cases of the exact-sum construction."""
    rng = np.random.default_rng(9600 + chunk)
    for case in range(12):
        M = int(rng.choice([1, 5, 64, 127, 128, 129, 200, 256, 300, 513, 700, 1024]))
        N = 8 * int(rng.integers(1, 160))
        K = 32 * int(rng.integers(1, 40))
        variant = VARIANTS[int(rng.integers(0, len(VARIANTS)))] if rng.integers(0, 4) else None
        nb = K // 32
        Xq, Wq = small_codes(rng.integers(1 << 30), (M, K)), small_codes(rng.integers(1 << 30), (N, K))
        ex = rng.integers(126, 129, size=(M, nb), dtype=np.uint8)
        ew = rng.integers(125, 128, size=(N, nb), dtype=np.uint8)
        b = inputs.small_int_bf16(961 + case, "bias", (N,), -4, 4) if rng.integers(0, 2) else None
        R = inputs.small_int_bf16(962 + case, "R", (M, N), -8, 8) if rng.integers(0, 2) else None
        inplace = R is not None and bool(rng.integers(0, 2))
        ref = oracle.outproj_mx(Xq, ex, Wq, ew, b, R)
        y = run_proj(Xq, ex, Wq, ew, b, R.copy() if inplace else R, inplace=inplace, variant=variant)
        ok, msg = kt.gate_exact(y, ref)
        assert ok, (M, N, K, variant, b is not None, R is not None, inplace, msg)


def test_mx_projection_exact_with_small_integer_epilogue():
    M, N, K = 600, 776, 96
    vals = np.array([0x00, 0x38, 0xB8], dtype=np.uint8)                     # 0, +-1
    rng = np.random.default_rng(910)
    Xq, Wq = vals[rng.integers(0, 3, (M, K))], vals[rng.integers(0, 3, (N, K))]
    ex = rng.integers(127, 129, size=(M, 3), dtype=np.uint8)
    ew = np.full((N, 3), 127, np.uint8)
    b = inputs.small_int_bf16(912, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(912, "R", (M, N), -8, 8)
    y = run_proj(Xq, ex, Wq, ew, b, R)
    ok, msg = kt.gate_exact(y, oracle.outproj_mx(Xq, ex, Wq, ew, b, R))
    assert ok, msg
    assert np.array_equal(run_proj(Xq, ex, Wq, ew, b, R.copy(), inplace=True), y)


@pytest.mark.parametrize("M,N,K", [(300, 520, 288), (1000, 776, 1056), (2500, 3080, 4096)])
def test_mx_projection_realistic_codes(M, N, K):
    """Codes and scales of normal data (with a per-block spread of magnitudes), bias and residual."""
    Xf = inputs.bf16_bits_to_f32(inputs.normal_bf16(920 + M, "X", (M, K), 1.0))
    Xf *= (2.0 ** np.random.default_rng(921).integers(-6, 7, size=(M, K // 32))).repeat(32, axis=1).astype(np.float32)
    Xq, ex = oracle.quantize_rows_mx(inputs.f32_to_bf16_bits(Xf))
    Wq, ew = oracle.quantize_rows_mx(inputs.normal_bf16(922, "W", (N, K), 1.0 / np.sqrt(K)))
    b = inputs.normal_bf16(924, "bias", (N,), 0.1)
    R = inputs.normal_bf16(924, "R", (M, N), 1.0)
    y = run_proj(Xq, ex, Wq, ew, b, R)
    ref = oracle.outproj_mx(Xq, ex, Wq, ew, b, R)
    ok, msg = kt.gate_a(y, ref)
    assert ok, msg
    assert kt.rel_fro(y, ref) <= 2.0 ** -8
    y0 = run_proj(Xq, ex, Wq, ew)
    assert kt.rel_fro(y0, oracle.outproj_mx(Xq, ex, Wq, ew)) <= 2.0 ** -8
    assert np.array_equal(run_proj(Xq, ex, Wq, ew, b, R), y)


def test_mx_quantise_then_project_on_device():
    """Both steps on the device, scales never leaving it: BF16 X, W -> code books -> projection, checked
    against the oracle's projection of the oracle's code books (the code books are bit-identical)."""
    M, N, K = 700, 1160, 2048
    X = inputs.normal_bf16(930, "X", (M, K), 1.0)
    W = inputs.normal_bf16(931, "W", (N, K), 1.0 / np.sqrt(K))
    R = inputs.normal_bf16(932, "R", (M, N), 1.0)
    Xq = torch.empty((M, K), dtype=torch.uint8, device="cuda").view(F8)
    Wq = torch.empty((N, K), dtype=torch.uint8, device="cuda").view(F8)
    SFX = torch.empty((kx.kx_mx_scale_bytes(M, K),), dtype=torch.uint8, device="cuda")
    SFW = torch.empty((kx.kx_mx_scale_bytes(N, K),), dtype=torch.uint8, device="cuda")
    kx.kx_quantize_rows_mxfp8(kt.to_dev(X), Xq, SFX)
    kx.kx_quantize_rows_mxfp8(kt.to_dev(W), Wq, SFW)
    Y = kt.nan_filled(M, N)
    kx.kx_outproj_residual_mxfp8(Xq, SFX, Wq, SFW, None, kt.to_dev(R), Y)
    status_ok()
    xq, ex = oracle.quantize_rows_mx(X)
    wq, ew = oracle.quantize_rows_mx(W)
    assert np.array_equal(host8(Xq), xq) and np.array_equal(SFW.cpu().numpy(), chunked(ew, K))
    ref = oracle.outproj_mx(xq, ex, wq, ew, None, R)
    ok, msg = kt.gate_a(kt.from_dev(Y), ref)
    assert ok, msg
    assert kt.rel_fro(kt.from_dev(Y), ref) <= 2.0 ** -8
    # and the quantised product stays close to the BF16 product it stands for
    exact = oracle.outproj(X, W, None, R)
    assert kt.rel_fro(kt.from_dev(Y), exact) <= 0.05


def test_mx_edges_and_argument_checks():
    Xq, Wq = small_codes(1, (8, 64)), small_codes(2, (16, 64))
    ex, ew = np.full((8, 2), 127, np.uint8), np.full((16, 2), 127, np.uint8)
    R = inputs.small_int_bf16(5, "R", (8, 16), -8, 8)
    b = inputs.small_int_bf16(5, "bias", (16,), -4, 4)
    # K = 0: Y = bias + R
    Y = kt.nan_filled(8, 16)
    bd, Rd = kt.to_dev(b), kt.to_dev(R)
    rc = kx.load().kx_outproj_residual_mxfp8(None, None, None, None, bd.data_ptr(), Rd.data_ptr(),
                                             Y.data_ptr(), 8, 16, 0, None)
    assert rc == kx.KX_OK
    torch.cuda.synchronize()
    ok, msg = kt.gate_exact(kt.from_dev(Y), oracle.outproj_mx(Xq[:, :0], ex[:, :0], Wq[:, :0], ew[:, :0], b, R))
    assert ok, msg
    lib = kx.load()
    x, w, sx, sw = dev8(Xq), dev8(Wq), dev(chunked(ex, 64)), dev(chunked(ew, 64))
    args = lambda **k: [k.get("x", x.data_ptr()), k.get("sx", sx.data_ptr()), k.get("w", w.data_ptr()),
                        k.get("sw", sw.data_ptr()), None, None, k.get("y", Y.data_ptr()),
                        k.get("M", 8), k.get("N", 16), k.get("K", 64), None]
    assert lib.kx_outproj_residual_mxfp8(*args(M=0)) == kx.KX_OK
    assert lib.kx_outproj_residual_mxfp8(*args(K=48)) == kx.KX_ERR_SHAPE
    assert lib.kx_outproj_residual_mxfp8(*args(N=12)) == kx.KX_ERR_SHAPE
    assert lib.kx_outproj_residual_mxfp8(*args(sx=None)) == kx.KX_ERR_NULL
    assert lib.kx_outproj_residual_mxfp8(*args(w=w.data_ptr() + 8)) == kx.KX_ERR_ALIGN
    assert lib.kx_outproj_residual_mxfp8(*args(y=x.data_ptr())) == kx.KX_ERR_OVERLAP
    ov = kx.make_override(block_n=64)
    assert lib.kx_outproj_residual_mxfp8_ex(*args(), ov) == kx.KX_ERR_PLAN
    A = kt.to_dev(inputs.normal_bf16(3, "X", (8, 64), 1.0))
    Q = torch.empty((8, 64), dtype=torch.uint8, device="cuda")
    SF = torch.empty((512,), dtype=torch.uint8, device="cuda")
    assert lib.kx_quantize_rows_mxfp8(A.data_ptr(), Q.data_ptr(), SF.data_ptr(), 8, 48, None) == kx.KX_ERR_SHAPE
    assert lib.kx_quantize_rows_mxfp8(A.data_ptr(), None, SF.data_ptr(), 8, 64, None) == kx.KX_ERR_NULL
    assert lib.kx_quantize_rows_mxfp8(A.data_ptr(), A.data_ptr(), SF.data_ptr(), 8, 64, None) == kx.KX_ERR_OVERLAP
    assert lib.kx_quantize_rows_mxfp8(A.data_ptr(), Q.data_ptr(), SF.data_ptr(), 0, 64, None) == kx.KX_OK
    assert lib.kx_quantize_rows_mxfp8(A.data_ptr(), Q.data_ptr(), SF.data_ptr(), 1, 32768 + 32, None) == kx.KX_ERR_SHAPE
    assert lib.kx_rmsnorm_quantize_mxfp8(A.data_ptr(), None, 1e-6, Q.data_ptr(), SF.data_ptr(), 8, 64, None) == kx.KX_ERR_NULL
    status_ok()


@pytest.mark.parametrize("M,N,K", [(4096, 4096, 4096), (16384, 4096, 14336)])
def test_mx_projection_full_sizes_sampled_rows(M, N, K):
    """The two projection shapes bench.py times for the block-scaled kind, in that launch configuration:
    exact on the small-value construction (block scales {1/2, 1} x {1/4, 1/2}: every partial sum stays an
    exactly representable multiple of 2^-5), then device-made code books of normal data with a residual
    within the gates; sampled rows."""
    rng = np.random.default_rng(980)
    nb = K // 32
    Xq, Wq = small_codes(981, (M, K)), small_codes(982, (N, K))
    ex = rng.integers(126, 128, size=(M, nb), dtype=np.uint8)
    ew = rng.integers(125, 127, size=(N, nb), dtype=np.uint8)
    rows = inputs.sampled_rows(M)[::8]
    Y = kt.nan_filled(M, N)
    kx.kx_outproj_residual_mxfp8(dev8(Xq), dev(chunked(ex, K)), dev8(Wq), dev(chunked(ew, K)), None, None, Y)
    status_ok()
    y = kt.from_dev(Y)
    assert not np.isnan(oracle.widen_bf16(y)).any()
    ok, msg = kt.gate_exact(y[rows], oracle.outproj_mx(Xq, ex, Wq, ew, rows=rows))
    assert ok, msg
    X = inputs.normal_bf16(983, "X", (M, K), 1.0)
    W = inputs.normal_bf16(984, "W", (N, K), 1.0 / np.sqrt(K))
    R = inputs.normal_bf16(985, "R", (M, N), 1.0)
    Xd = torch.empty((M, K), dtype=torch.uint8, device="cuda").view(F8)
    Wd = torch.empty((N, K), dtype=torch.uint8, device="cuda").view(F8)
    SFX = torch.empty((kx.kx_mx_scale_bytes(M, K),), dtype=torch.uint8, device="cuda")
    SFW = torch.empty((kx.kx_mx_scale_bytes(N, K),), dtype=torch.uint8, device="cuda")
    kx.kx_quantize_rows_mxfp8(kt.to_dev(X), Xd, SFX)
    kx.kx_quantize_rows_mxfp8(kt.to_dev(W), Wd, SFW)
    kx.kx_outproj_residual_mxfp8(Xd, SFX, Wd, SFW, None, kt.to_dev(R), Y)
    status_ok()
    y = kt.from_dev(Y)
    xq, ex2 = oracle.quantize_rows_mx(X)
    wq, ew2 = oracle.quantize_rows_mx(W)
    assert np.array_equal(host8(Xd)[rows], xq[rows]) and np.array_equal(SFW.cpu().numpy(), chunked(ew2, K))
    ref = oracle.outproj_mx(xq, ex2, wq, ew2, None, R, rows=rows)
    ok, msg = kt.gate_a(y[rows], ref)
    assert ok, msg
    assert kt.rel_fro(y[rows], ref) <= 2.0 ** -8


# ------------------------------------------------------------------ gate/up + SwiGLU
def run_swiglu(Xq, ex, Wgq, eg, Wuq, eu):
    (M, K), I = Xq.shape, Wgq.shape[0]
    Z = kt.nan_filled(M, I)
    sfgu = np.concatenate([chunked(eg, K), chunked(eu, K)])
    kx.kx_gate_up_swiglu_mxfp8(dev8(Xq), dev(chunked(ex, K)), dev8(Wgq), dev8(Wuq), dev(sfgu), Z)
    status_ok()
    return kt.from_dev(Z)


def check_swiglu(z_bits, ref):
    ok, msg = kt.gate_a(z_bits, ref)
    assert ok, msg
    assert kt.rel_fro(z_bits, ref) <= 2.0 ** -8
    z = oracle.widen_bf16(z_bits)
    assert (np.abs(z - ref) <= 2.0 ** -7 * np.abs(ref) + 2e-3).all()


@pytest.mark.parametrize("M,I,K", [(128, 128, 128), (300, 520, 288), (640, 1024, 512), (7, 776, 1120),
                                   (2048, 4096, 512), (2500, 3080, 288)])
def test_mx_swiglu_matches_oracle(M, I, K):
    Xq, ex = oracle.quantize_rows_mx(inputs.normal_bf16(990 + M, "X", (M, K), 1.0))
    Wgq, eg = oracle.quantize_rows_mx(inputs.normal_bf16(991, "W", (I, K), 1.0 / np.sqrt(K)))
    Wuq, eu = oracle.quantize_rows_mx(inputs.normal_bf16(992, "W", (I, K), 1.0 / np.sqrt(K)))
    check_swiglu(run_swiglu(Xq, ex, Wgq, eg, Wuq, eu), oracle.swiglu_mx(Xq, ex, Wgq, eg, Wuq, eu))


def test_mx_swiglu_exact_pins_and_pairing():
    """u = 1 exactly (one-hot up rows) leaves silu(g) for an exactly representable g; one-hot gate rows select
    which up row pairs with which gate row; the scale arrays of gate and up are not interchangeable."""
    M, I, K = 130, 264, 64
    rng = np.random.default_rng(993)
    Xq = small_codes(994, (M, K))
    Xq[:, 0] = 0x38                                            # x[:, 0] = 1
    ex = np.full((M, 2), 127, np.uint8)
    Wgq = small_codes(995, (I, K))
    eg = rng.integers(124, 127, size=(I, 2), dtype=np.uint8)
    Wuq = np.zeros((I, K), np.uint8)
    Wuq[:, 0] = 0x38                                           # u = 1 * 2^(eu - 127)
    eu = rng.integers(127, 130, size=(I, 2), dtype=np.uint8)
    z = run_swiglu(Xq, ex, Wgq, eg, Wuq, eu)
    ref = oracle.swiglu_mx(Xq, ex, Wgq, eg, Wuq, eu)
    check_swiglu(z, ref)
    g = oracle.outproj_mx(Xq, ex, Wgq, eg)
    assert np.allclose(ref, g / (1 + np.exp(-g)) * (2.0 ** (eu[:, 0].astype(np.float64) - 127))[None, :])
    assert np.abs(ref).max() > 1.0
    # swapping the two halves of the scale array changes the result
    Z = kt.nan_filled(M, I)
    sfug = np.concatenate([chunked(eu, K), chunked(eg, K)])
    kx.kx_gate_up_swiglu_mxfp8(dev8(Xq), dev(chunked(ex, K)), dev8(Wgq), dev8(Wuq), dev(sfug), Z)
    assert not np.array_equal(kt.from_dev(Z), z)


def test_mx_gate_up_code_books_and_chain_on_device():
    """Code books of both weight matrices in the layout the GEMM reads, then RMSNorm + code book -> gate/up + SwiGLU
    on the device, against the oracle on the oracle's code books (bit-identical to the device's)."""
    M, I, K = 520, 1160, 1024
    H = inputs.normal_bf16(996, "R", (M, K), 1.3)
    gam = inputs.normal_bf16(996, "bias", (K,), 1.0)
    Wg = inputs.normal_bf16(997, "W", (I, K), 1.0 / np.sqrt(K))
    Wu = inputs.normal_bf16(998, "W", (I, K), 1.0 / np.sqrt(K))
    f8 = lambda *shape: torch.empty(shape, dtype=torch.uint8, device="cuda").view(F8)
    Qg, Qu, Xq = f8(I, K), f8(I, K), f8(M, K)
    SFGU = torch.full((2 * kx.kx_mx_scale_bytes(I, K),), 0xEE, dtype=torch.uint8, device="cuda")
    SFX = torch.empty((kx.kx_mx_scale_bytes(M, K),), dtype=torch.uint8, device="cuda")
    kx.kx_quantize_gate_up_mxfp8(kt.to_dev(Wg), kt.to_dev(Wu), Qg, Qu, SFGU)
    Zn = kt.nan_filled(M, K)
    kx.kx_rmsnorm(kt.to_dev(H), kt.to_dev(gam), 1e-6, Zn)
    kx.kx_rmsnorm_quantize_mxfp8(kt.to_dev(H), kt.to_dev(gam), 1e-6, Xq, SFX)
    Z = kt.nan_filled(M, I)
    kx.kx_gate_up_swiglu_mxfp8(Xq, SFX, Qg, Qu, SFGU, Z)
    status_ok()
    qg, eg = oracle.quantize_rows_mx(Wg)
    qu, eu = oracle.quantize_rows_mx(Wu)
    xq, ex = oracle.quantize_rows_mx(kt.from_dev(Zn))
    assert np.array_equal(host8(Qg), qg) and np.array_equal(host8(Qu), qu) and np.array_equal(host8(Xq), xq)
    assert np.array_equal(SFGU.cpu().numpy(), np.concatenate([chunked(eg, K), chunked(eu, K)]))
    check_swiglu(kt.from_dev(Z), oracle.swiglu_mx(xq, ex, qg, eg, qu, eu))


def test_mx_swiglu_full_size_sampled_rows():
    """The gate/up shape of the benchmark (M = 4096 tokens, I = 14336, K = 4096) on sampled rows."""
    M, I, K = 4096, 14336, 4096
    Xq, ex = oracle.quantize_rows_mx(inputs.normal_bf16(999, "X", (M, K), 1.0))
    Wgq, eg = oracle.quantize_rows_mx(inputs.normal_bf16(1000, "W", (I, K), 1.0 / np.sqrt(K)))
    Wuq, eu = oracle.quantize_rows_mx(inputs.normal_bf16(1001, "W", (I, K), 1.0 / np.sqrt(K)))
    rows = inputs.sampled_rows(M)[::8]
    z = run_swiglu(Xq, ex, Wgq, eg, Wuq, eu)
    assert not np.isnan(oracle.widen_bf16(z)).any()
    check_swiglu(z[rows], oracle.swiglu_mx(Xq, ex, Wgq, eg, Wuq, eu, rows=rows))
