"""4-bit block-scaled branch: the code book (packed codes and chunked scale bytes) bit for bit, the
projection bit for bit where every partial sum is exactly representable, the rest within the
tolerance gates of the BF16 path."""
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


def chunked(S, cols):
    """Row-major scale bytes [rows, cols / 16] -> the library's chunked array (index arithmetic only; padding 0)."""
    rows, nb = S.shape
    rc, kc = (rows + 127) // 128, (cols + 63) // 64
    out = np.zeros((rc, kc, 32, 4, 4), dtype=np.uint8)
    r = np.arange(rows)[:, None]
    j = np.arange(nb)[None, :]
    out[r // 128, j // 4, r % 32, (r % 128) // 32, j % 4] = S
    return out.reshape(-1)


def gpu_quantize(A, gs):
    rows, cols = A.shape
    Q = torch.full((rows, cols // 2), 0x55, dtype=torch.uint8, device="cuda")
    SF = torch.full((kx.kx_nvfp4_scale_bytes(rows, cols),), 0xEE, dtype=torch.uint8, device="cuda")
    kx.kx_quantize_rows_nvfp4(kt.to_dev(A), gs, Q, SF)
    return Q.cpu().numpy(), SF.cpu().numpy()


def test_scale_bytes():
    assert kx.kx_nvfp4_scale_bytes(1, 16) == 512 and kx.kx_nvfp4_scale_bytes(128, 64) == 512
    assert kx.kx_nvfp4_scale_bytes(129, 80) == 4 * 512 and kx.kx_nvfp4_scale_bytes(-1, 64) < 0


@pytest.mark.parametrize("rows,cols", [(1, 16), (5, 80), (300, 2064), (129, 4096), (3, 32768), (700, 1024), (7, 3072), (5, 2560), (9, 7168), (5, 6144), (9000, 256)])
def test_nvfp4_code_book_bit_exact(rows, cols):
    A = inputs.normal_bf16(1000 + cols, "X", (rows, cols), 2.5)
    f = inputs.bf16_bits_to_f32(A)
    f[0, :16] *= 2.0 ** -12
    if cols >= 48:
        f[0, 16:32] *= 40.0
        f[0, 32:48] = 0
    if rows > 2:
        f[1] = 0
    A = inputs.f32_to_bf16_bits(f)
    gs = float(np.float32(np.abs(inputs.bf16_bits_to_f32(A)).max() / (448.0 * 6.0)))
    Q, SF = gpu_quantize(A, gs)
    Qr, Sr = oracle.quantize_rows_nvfp4(A, gs)
    assert np.array_equal(SF, chunked(Sr, cols))
    assert np.array_equal(Q, Qr)


def test_nvfp4_code_book_grid_ties():
    vals = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    row = np.concatenate([vals, -vals, np.r_[6.0, mids], np.r_[-6.0, -mids, np.zeros(0)], np.zeros(0)])
    row = np.concatenate([row, np.zeros(32 - len(row))]).reshape(1, 32)
    A = inputs.f32_to_bf16_bits(row.astype(np.float32))
    Q, SF = gpu_quantize(A, 1.0)
    Qr, Sr = oracle.quantize_rows_nvfp4(A, 1.0)
    assert np.array_equal(Q, Qr) and np.array_equal(SF, chunked(Sr, 32))
    lo, hi = Q[0] & 15, Q[0] >> 4
    codes = np.stack([lo, hi], 1).reshape(-1)
    assert codes[:8].tolist() == list(range(8)) and codes[17:24].tolist() == [0, 2, 2, 4, 4, 6, 6]


# ------------------------------------------------------------------ projection
def pack(codes):
    return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)


def small_codes(seed, shape):
    """E2M1 codes of {0, +-0.5, +-1, +-2, +-4}"""
    pool = np.array([0, 1, 2, 4, 6, 9, 10, 12, 14], dtype=np.uint8)
    return pool[np.random.default_rng(seed).integers(0, len(pool), size=shape)]


VARIANTS = [128, 192, 256]


def run_proj(Xq, sx, Wq, sw, alpha, b=None, R=None, inplace=False, variant=None):
    M, N, K = Xq.shape[0], Wq.shape[0], Xq.shape[1] * 2
    ov = None if variant is None else kx.make_override(block_n=variant)
    if inplace:
        Y = kt.to_dev(R)
        Rd = Y
    else:
        Y = kt.nan_filled(M, N)
        Rd = kt.to_dev(R)
    kx.kx_outproj_residual_nvfp4(dev(Xq), dev(chunked(sx, K)), dev(Wq), dev(chunked(sw, K)), alpha, kt.to_dev(b), Rd, Y,
                                 override=ov)
    status_ok()
    return kt.from_dev(Y)


@pytest.mark.parametrize("variant", [None] + VARIANTS)
@pytest.mark.parametrize("M,N,K", [(128, 128, 256), (300, 520, 288), (1000, 776, 1056), (7, 64, 32), (260, 960, 384),
                                   (2500, 3080, 416), (640, 1024, 4096)])
def test_nvfp4_projection_exact_on_small_values(variant, M, N, K):
    """Element values in {0, +-0.5, +-1, +-2, +-4}, block scales in {0.5, 1, 2} (A) and {0.25, 0.5, 1} (B) per
    (row, 16-element block), alpha = 0.5: every product is a multiple of 2^-5 of size at most 32 and every
    partial sum is exactly representable, so any accumulation order gives the exact sum - and a scale read
    from the wrong row, block or byte changes it."""
    rng = np.random.default_rng(1100 + M + N + K)
    nb = K // 16
    Xq, Wq = pack(small_codes(1101 + M, (M, K))), pack(small_codes(1102 + N, (N, K)))
    sx = np.array([0x30, 0x38, 0x40], np.uint8)[rng.integers(0, 3, size=(M, nb))]
    sw = np.array([0x28, 0x30, 0x38], np.uint8)[rng.integers(0, 3, size=(N, nb))]
    b = inputs.small_int_bf16(1103, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(1103, "R", (M, N), -8, 8)
    ok, msg = kt.gate_exact(run_proj(Xq, sx, Wq, sw, 0.5, b, R, variant=variant), oracle.outproj_nvfp4(Xq, sx, Wq, sw, 0.5, b, R))
    assert ok, msg


@pytest.mark.parametrize("chunk", range(3))
def test_nvfp4_random_shapes_and_tile_shapes_are_exact(chunk):
    """Seeded random (M, N, K, tile shape, bias / residual / in place) cases of the exact-sum construction."""
    rng = np.random.default_rng(9700 + chunk)
    for case in range(12):
        M = int(rng.choice([1, 5, 64, 127, 128, 129, 200, 256, 300, 513, 700, 1024]))
        N = 8 * int(rng.integers(1, 160))
        K = 32 * int(rng.integers(1, 40))
        variant = VARIANTS[int(rng.integers(0, len(VARIANTS)))] if rng.integers(0, 4) else None
        nb = K // 16
        Xq, Wq = pack(small_codes(rng.integers(1 << 30), (M, K))), pack(small_codes(rng.integers(1 << 30), (N, K)))
        sx = np.array([0x30, 0x38, 0x40], np.uint8)[rng.integers(0, 3, size=(M, nb))]
        sw = np.array([0x28, 0x30, 0x38], np.uint8)[rng.integers(0, 3, size=(N, nb))]
        b = inputs.small_int_bf16(971 + case, "bias", (N,), -4, 4) if rng.integers(0, 2) else None
        R = inputs.small_int_bf16(972 + case, "R", (M, N), -8, 8) if rng.integers(0, 2) else None
        inplace = R is not None and bool(rng.integers(0, 2))
        alpha = float(rng.choice([0.25, 0.5, 1.0, 2.0]))
        ref = oracle.outproj_nvfp4(Xq, sx, Wq, sw, alpha, b, R)
        y = run_proj(Xq, sx, Wq, sw, alpha, b, R.copy() if inplace else R, inplace=inplace, variant=variant)
        ok, msg = kt.gate_exact(y, ref)
        assert ok, (M, N, K, variant, alpha, b is not None, R is not None, inplace, msg)


@pytest.mark.parametrize("M,N,K", [(300, 520, 288), (1000, 776, 1056), (2500, 3080, 4096)])
def test_nvfp4_projection_realistic_codes(M, N, K):
    X = inputs.normal_bf16(1120 + M, "X", (M, K), 1.0)
    W = inputs.normal_bf16(1121, "W", (N, K), 1.0 / np.sqrt(K))
    gsx = float(np.float32(np.abs(inputs.bf16_bits_to_f32(X)).max() / 2688.0))
    gsw = float(np.float32(np.abs(inputs.bf16_bits_to_f32(W)).max() / 2688.0))
    Xq, sx = oracle.quantize_rows_nvfp4(X, gsx)
    Wq, sw = oracle.quantize_rows_nvfp4(W, gsw)
    alpha = float(np.float32(gsx) * np.float32(gsw))
    b = inputs.normal_bf16(1124, "bias", (N,), 0.1)
    R = inputs.normal_bf16(1124, "R", (M, N), 1.0)
    y = run_proj(Xq, sx, Wq, sw, alpha, b, R)
    ref = oracle.outproj_nvfp4(Xq, sx, Wq, sw, alpha, b, R)
    ok, msg = kt.gate_a(y, ref)
    assert ok, msg
    assert kt.rel_fro(y, ref) <= 2.0 ** -8
    y0 = run_proj(Xq, sx, Wq, sw, alpha)
    assert kt.rel_fro(y0, oracle.outproj_nvfp4(Xq, sx, Wq, sw, alpha)) <= 2.0 ** -8
    assert np.array_equal(run_proj(Xq, sx, Wq, sw, alpha, b, R), y)
    assert np.array_equal(run_proj(Xq, sx, Wq, sw, alpha, b, R.copy(), inplace=True), y)


def test_nvfp4_quantise_then_project_on_device():
    M, N, K = 700, 1160, 2048
    X = inputs.normal_bf16(1130, "X", (M, K), 1.0)
    W = inputs.normal_bf16(1131, "W", (N, K), 1.0 / np.sqrt(K))
    R = inputs.normal_bf16(1132, "R", (M, N), 1.0)
    gsx = float(np.float32(np.abs(inputs.bf16_bits_to_f32(X)).max() / 2688.0))
    gsw = float(np.float32(np.abs(inputs.bf16_bits_to_f32(W)).max() / 2688.0))
    Xq = torch.empty((M, K // 2), dtype=torch.uint8, device="cuda")
    Wq = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
    SFX = torch.empty((kx.kx_nvfp4_scale_bytes(M, K),), dtype=torch.uint8, device="cuda")
    SFW = torch.empty((kx.kx_nvfp4_scale_bytes(N, K),), dtype=torch.uint8, device="cuda")
    kx.kx_quantize_rows_nvfp4(kt.to_dev(X), gsx, Xq, SFX)
    kx.kx_quantize_rows_nvfp4(kt.to_dev(W), gsw, Wq, SFW)
    Y = kt.nan_filled(M, N)
    alpha = float(np.float32(gsx) * np.float32(gsw))
    kx.kx_outproj_residual_nvfp4(Xq, SFX, Wq, SFW, alpha, None, kt.to_dev(R), Y)
    status_ok()
    xq, sx = oracle.quantize_rows_nvfp4(X, gsx)
    wq, sw = oracle.quantize_rows_nvfp4(W, gsw)
    assert np.array_equal(Xq.cpu().numpy(), xq) and np.array_equal(SFW.cpu().numpy(), chunked(sw, K))
    ref = oracle.outproj_nvfp4(xq, sx, wq, sw, alpha, None, R)
    ok, msg = kt.gate_a(kt.from_dev(Y), ref)
    assert ok, msg
    assert kt.rel_fro(kt.from_dev(Y), ref) <= 2.0 ** -8
    assert kt.rel_fro(kt.from_dev(Y), oracle.outproj(X, W, None, R)) <= 0.15      # 4-bit operands: coarse but close


def test_nvfp4_edges_and_argument_checks():
    lib = kx.load()
    Xq, Wq = pack(small_codes(1, (8, 64))), pack(small_codes(2, (16, 64)))
    sx, sw = np.full((8, 4), 0x38, np.uint8), np.full((16, 4), 0x38, np.uint8)
    R = inputs.small_int_bf16(5, "R", (8, 16), -8, 8)
    b = inputs.small_int_bf16(5, "bias", (16,), -4, 4)
    Y = kt.nan_filled(8, 16)
    bd, Rd = kt.to_dev(b), kt.to_dev(R)
    assert lib.kx_outproj_residual_nvfp4(None, None, None, None, 1.0, bd.data_ptr(), Rd.data_ptr(), Y.data_ptr(), 8, 16, 0,
                                         None, None) == kx.KX_OK
    torch.cuda.synchronize()
    ok, msg = kt.gate_exact(kt.from_dev(Y), oracle.outproj_nvfp4(Xq[:, :0], sx[:, :0], Wq[:, :0], sw[:, :0], 1.0, b, R))
    assert ok, msg
    x, w, fx, fw = dev(Xq), dev(Wq), dev(chunked(sx, 64)), dev(chunked(sw, 64))
    args = lambda **k: [k.get("x", x.data_ptr()), k.get("fx", fx.data_ptr()), k.get("w", w.data_ptr()), fw.data_ptr(), 1.0,
                        None, None, k.get("y", Y.data_ptr()), k.get("M", 8), k.get("N", 16), k.get("K", 64), None, None]
    assert lib.kx_outproj_residual_nvfp4(*args(M=0)) == kx.KX_OK
    assert lib.kx_outproj_residual_nvfp4(*args(K=48)) == kx.KX_ERR_SHAPE
    assert lib.kx_outproj_residual_nvfp4(*args(N=12)) == kx.KX_ERR_SHAPE
    assert lib.kx_outproj_residual_nvfp4(*args(fx=None)) == kx.KX_ERR_NULL
    assert lib.kx_outproj_residual_nvfp4(*args(w=w.data_ptr() + 8)) == kx.KX_ERR_ALIGN
    assert lib.kx_outproj_residual_nvfp4(*args(y=x.data_ptr())) == kx.KX_ERR_OVERLAP
    A = kt.to_dev(inputs.normal_bf16(3, "X", (8, 64), 1.0))
    Q = torch.empty((8, 32), dtype=torch.uint8, device="cuda")
    SF = torch.empty((512,), dtype=torch.uint8, device="cuda")
    assert lib.kx_quantize_rows_nvfp4(A.data_ptr(), 1.0, Q.data_ptr(), SF.data_ptr(), 8, 40, None) == kx.KX_ERR_SHAPE
    assert lib.kx_quantize_rows_nvfp4(A.data_ptr(), 0.0, Q.data_ptr(), SF.data_ptr(), 8, 64, None) == kx.KX_ERR_SHAPE
    assert lib.kx_quantize_rows_nvfp4(A.data_ptr(), 1.0, None, SF.data_ptr(), 8, 64, None) == kx.KX_ERR_NULL
    assert lib.kx_quantize_rows_nvfp4(A.data_ptr(), 1.0, Q.data_ptr(), SF.data_ptr(), 0, 64, None) == kx.KX_OK
    status_ok()


@pytest.mark.parametrize("M,N,K", [(4096, 4096, 4096), (16384, 4096, 14336)])
def test_nvfp4_projection_full_sizes_sampled_rows(M, N, K):
    """The two projection shapes bench.py times for the 4-bit kind, in that launch configuration: exact on
    the small-value construction (block scales {1/2, 1} x {1/4, 1/2}), then device-made code books of normal
    data with a residual within the gates; sampled rows."""
    rng = np.random.default_rng(1180)
    nb = K // 16
    Xq, Wq = pack(small_codes(1181, (M, K))), pack(small_codes(1182, (N, K)))
    sx = np.array([0x30, 0x38], np.uint8)[rng.integers(0, 2, size=(M, nb))]
    sw = np.array([0x28, 0x30], np.uint8)[rng.integers(0, 2, size=(N, nb))]
    rows = inputs.sampled_rows(M)[::8]
    Y = kt.nan_filled(M, N)
    kx.kx_outproj_residual_nvfp4(dev(Xq), dev(chunked(sx, K)), dev(Wq), dev(chunked(sw, K)), 1.0, None, None, Y)
    status_ok()
    y = kt.from_dev(Y)
    assert not np.isnan(oracle.widen_bf16(y)).any()
    ok, msg = kt.gate_exact(y[rows], oracle.outproj_nvfp4(Xq, sx, Wq, sw, 1.0, rows=rows))
    assert ok, msg
    X = inputs.normal_bf16(1183, "X", (M, K), 1.0)
    W = inputs.normal_bf16(1184, "W", (N, K), 1.0 / np.sqrt(K))
    R = inputs.normal_bf16(1185, "R", (M, N), 1.0)
    gsx = float(np.float32(np.abs(inputs.bf16_bits_to_f32(X)).max() / 2688.0))
    gsw = float(np.float32(np.abs(inputs.bf16_bits_to_f32(W)).max() / 2688.0))
    alpha = float(np.float32(gsx) * np.float32(gsw))
    Xd = torch.empty((M, K // 2), dtype=torch.uint8, device="cuda")
    Wd = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
    SFX = torch.empty((kx.kx_nvfp4_scale_bytes(M, K),), dtype=torch.uint8, device="cuda")
    SFW = torch.empty((kx.kx_nvfp4_scale_bytes(N, K),), dtype=torch.uint8, device="cuda")
    kx.kx_quantize_rows_nvfp4(kt.to_dev(X), gsx, Xd, SFX)
    kx.kx_quantize_rows_nvfp4(kt.to_dev(W), gsw, Wd, SFW)
    kx.kx_outproj_residual_nvfp4(Xd, SFX, Wd, SFW, alpha, None, kt.to_dev(R), Y)
    status_ok()
    y = kt.from_dev(Y)
    xq, sx2 = oracle.quantize_rows_nvfp4(X, gsx)
    wq, sw2 = oracle.quantize_rows_nvfp4(W, gsw)
    assert np.array_equal(Xd.cpu().numpy()[rows], xq[rows]) and np.array_equal(SFW.cpu().numpy(), chunked(sw2, K))
    ref = oracle.outproj_nvfp4(xq, sx2, wq, sw2, alpha, None, R, rows=rows)
    ok, msg = kt.gate_a(y[rows], ref)
    assert ok, msg
    assert kt.rel_fro(y[rows], ref) <= 2.0 ** -8


# ------------------------------------------------------------------ RMSNorm-fused code book, gate/up + SwiGLU
@pytest.mark.parametrize("M,N", [(130, 4096), (1000, 5120), (9, 32768), (300, 1040), (7, 3072), (3, 8192), (5, 6144), (9, 7168), (5, 2560), (9000, 256)])
def test_nvfp4_rmsnorm_code_book(M, N):
    """Fused RMSNorm + code book = code book of the device's own BF16 RMSNorm output, bit for bit."""
    H = inputs.normal_bf16(1150 + N, "R", (M, N), 1.3)
    g = inputs.normal_bf16(1150 + N, "bias", (N,), 1.0)
    Z = kt.nan_filled(M, N)
    kx.kx_rmsnorm(kt.to_dev(H), kt.to_dev(g), 1e-6, Z)
    gs = 8.0 / 2688.0
    Q = torch.full((M, N // 2), 0x55, dtype=torch.uint8, device="cuda")
    SF = torch.full((kx.kx_nvfp4_scale_bytes(M, N),), 0xEE, dtype=torch.uint8, device="cuda")
    kx.kx_rmsnorm_quantize_nvfp4(kt.to_dev(H), kt.to_dev(g), 1e-6, gs, Q, SF)
    Qr, Sr = oracle.quantize_rows_nvfp4(kt.from_dev(Z), gs)
    assert np.array_equal(Q.cpu().numpy(), Qr) and np.array_equal(SF.cpu().numpy(), chunked(Sr, N))


def check_swiglu(z_bits, ref):
    ok, msg = kt.gate_a(z_bits, ref)
    assert ok, msg
    assert kt.rel_fro(z_bits, ref) <= 2.0 ** -8
    z = oracle.widen_bf16(z_bits)
    assert (np.abs(z - ref) <= 2.0 ** -7 * np.abs(ref) + 2e-3).all()


def run_swiglu(Xq, sx, Wgq, sg, Wuq, su, ag, au):
    M, I, K = Xq.shape[0], Wgq.shape[0], Xq.shape[1] * 2
    Z = kt.nan_filled(M, I)
    sfgu = np.concatenate([chunked(sg, K), chunked(su, K)])
    kx.kx_gate_up_swiglu_nvfp4(dev(Xq), dev(chunked(sx, K)), dev(Wgq), dev(Wuq), dev(sfgu), ag, au, Z)
    status_ok()
    return kt.from_dev(Z)


def codes_of(seed, name, shape, std):
    A = inputs.normal_bf16(seed, name, shape, std)
    gs = float(np.float32(np.abs(inputs.bf16_bits_to_f32(A)).max() / 2688.0))
    Q, S = oracle.quantize_rows_nvfp4(A, gs)
    return Q, S, gs


@pytest.mark.parametrize("M,I,K", [(128, 128, 256), (300, 520, 288), (640, 1024, 512), (7, 776, 1120),
                                   (2048, 4096, 512), (2500, 3080, 288)])
def test_nvfp4_swiglu_matches_oracle(M, I, K):
    Xq, sx, gx = codes_of(1160 + M, "X", (M, K), 1.0)
    Wgq, sg, gg = codes_of(1161, "W", (I, K), 1.0 / np.sqrt(K))
    Wuq, su, gu = codes_of(1162, "W", (I, K), 2.0 / np.sqrt(K))
    ag, au = float(np.float32(gx) * np.float32(gg)), float(np.float32(gx) * np.float32(gu))
    check_swiglu(run_swiglu(Xq, sx, Wgq, sg, Wuq, su, ag, au), oracle.swiglu_nvfp4(Xq, sx, Wgq, sg, Wuq, su, ag, au))


def test_nvfp4_gate_up_code_books_and_chain_on_device():
    M, I, K = 520, 1160, 1024
    H = inputs.normal_bf16(1170, "R", (M, K), 1.3)
    gam = inputs.normal_bf16(1170, "bias", (K,), 1.0)
    Wg = inputs.normal_bf16(1171, "W", (I, K), 1.0 / np.sqrt(K))
    Wu = inputs.normal_bf16(1172, "W", (I, K), 1.0 / np.sqrt(K))
    gsx, gsg, gsu = 8.0 / 2688.0, 0.2 / 2688.0, 0.25 / 2688.0
    u8 = lambda *shape: torch.empty(shape, dtype=torch.uint8, device="cuda")
    Qg, Qu, Xq = u8(I, K // 2), u8(I, K // 2), u8(M, K // 2)
    SFGU = torch.full((2 * kx.kx_nvfp4_scale_bytes(I, K),), 0xEE, dtype=torch.uint8, device="cuda")
    SFX = u8(kx.kx_nvfp4_scale_bytes(M, K))
    kx.kx_quantize_gate_up_nvfp4(kt.to_dev(Wg), kt.to_dev(Wu), gsg, gsu, Qg, Qu, SFGU)
    Zn = kt.nan_filled(M, K)
    kx.kx_rmsnorm(kt.to_dev(H), kt.to_dev(gam), 1e-6, Zn)
    kx.kx_rmsnorm_quantize_nvfp4(kt.to_dev(H), kt.to_dev(gam), 1e-6, gsx, Xq, SFX)
    Z = kt.nan_filled(M, I)
    ag, au = float(np.float32(gsx) * np.float32(gsg)), float(np.float32(gsx) * np.float32(gsu))
    kx.kx_gate_up_swiglu_nvfp4(Xq, SFX, Qg, Qu, SFGU, ag, au, Z)
    status_ok()
    qg, sg = oracle.quantize_rows_nvfp4(Wg, gsg)
    qu, su = oracle.quantize_rows_nvfp4(Wu, gsu)
    xq, sx = oracle.quantize_rows_nvfp4(kt.from_dev(Zn), gsx)
    assert np.array_equal(Qg.cpu().numpy(), qg) and np.array_equal(Qu.cpu().numpy(), qu) and np.array_equal(Xq.cpu().numpy(), xq)
    assert np.array_equal(SFGU.cpu().numpy(), np.concatenate([chunked(sg, K), chunked(su, K)]))
    check_swiglu(kt.from_dev(Z), oracle.swiglu_nvfp4(xq, sx, qg, sg, qu, su, ag, au))


def test_nvfp4_swiglu_full_size_sampled_rows():
    """The gate/up shape of the benchmark (M = 4096 tokens, I = 14336, K = 4096) on sampled rows."""
    M, I, K = 4096, 14336, 4096
    Xq, sx, gx = codes_of(1175, "X", (M, K), 1.0)
    Wgq, sg, gg = codes_of(1176, "W", (I, K), 1.0 / np.sqrt(K))
    Wuq, su, gu = codes_of(1177, "W", (I, K), 1.0 / np.sqrt(K))
    ag, au = float(np.float32(gx) * np.float32(gg)), float(np.float32(gx) * np.float32(gu))
    rows = inputs.sampled_rows(M)[::8]
    z = run_swiglu(Xq, sx, Wgq, sg, Wuq, su, ag, au)
    assert not np.isnan(oracle.widen_bf16(z)).any()
    check_swiglu(z[rows], oracle.swiglu_nvfp4(Xq, sx, Wgq, sg, Wuq, su, ag, au, rows=rows))
