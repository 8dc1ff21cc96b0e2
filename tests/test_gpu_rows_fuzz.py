"""Seeded random row counts and row lengths through the row kernels (RMSNorm, per-row and per-block code books,
plain and fused behind the normalisation): every thread-per-row / vectors-per-thread instantiation, rows that fill
their threads exactly and rows that do not, odd row counts (a row group left idle in the last step), enough rows
for the prefetch ring to wrap and for the non-persistent grid.  Codes and scales are compared bit for bit with the
oracle's code book of the device's own BF16 RMSNorm output; that output against the oracle's RMSNorm within one
BF16 rounding."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt
from test_gpu_mxfp8 import chunked as chunked_mx, host8
from test_gpu_nvfp4 import chunked as chunked_nv
from test_gpu_rmsnorm import gate_norm

pytestmark = pytest.mark.gpu
F8 = torch.float8_e4m3fn


def draw(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        N = 32 * int(rng.integers(1, 257))                      # 32 .. 8192: the short-row kernel
        if rng.random() < 0.1:
            N = 32 * int(rng.integers(257, 400))                # a few rows for the long-row kernels
        cap = max(1, min(6000, (1 << 21) // N))
        M = int(rng.integers(1, cap + 1))
        out.append((M, N))
    return out


@pytest.mark.parametrize("chunk", range(6))
def test_row_kernels_random_shapes(chunk):
    for (M, N) in draw(5, 4100 + chunk):
        H = inputs.normal_bf16(7000 + N + M, "R", (M, N), 1.7)
        g = inputs.normal_bf16(7000 + N + M, "bias", (N,), 1.0)
        Hd, gd = kt.to_dev(H), kt.to_dev(g)
        Z = kt.nan_filled(M, N)
        kx.kx_rmsnorm(Hd, gd, 1e-6, Z)
        z_bits = kt.from_dev(Z)
        gate_norm(z_bits, oracle.rmsnorm(H, g, 1e-6))
        # per-row INT8, fused and plain (plain: code book of H itself)
        Q = torch.full((M, N), 77, dtype=torch.int8, device="cuda")
        S = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
        kx.kx_rmsnorm_quantize_int8(Hd, gd, 1e-6, Q, S)
        Qr, Sr = oracle.quantize_rows(z_bits)
        assert np.array_equal(S.cpu().numpy(), Sr) and np.array_equal(Q.cpu().numpy(), Qr), (M, N)
        kx.kx_quantize_rows_int8(Hd, Q, S)
        Qr, Sr = oracle.quantize_rows(H)
        assert np.array_equal(S.cpu().numpy(), Sr) and np.array_equal(Q.cpu().numpy(), Qr), (M, N)
        # per-row FP8
        Q8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda").view(F8)
        kx.kx_rmsnorm_quantize_fp8(Hd, gd, 1e-6, Q8, S)
        Qr, Sr = oracle.quantize_rows_fp8(z_bits)
        assert np.array_equal(host8(Q8), Qr) and np.array_equal(S.cpu().numpy(), Sr), (M, N)
        # block-scaled FP8
        SF = torch.full((kx.kx_mx_scale_bytes(M, N),), 0xEE, dtype=torch.uint8, device="cuda")
        kx.kx_rmsnorm_quantize_mxfp8(Hd, gd, 1e-6, Q8, SF)
        Qr, Er = oracle.quantize_rows_mx(z_bits)
        assert np.array_equal(host8(Q8), Qr) and np.array_equal(SF.cpu().numpy(), chunked_mx(Er, N)), (M, N)
        kx.kx_quantize_rows_mxfp8(Hd, Q8, SF)
        Qr, Er = oracle.quantize_rows_mx(H)
        assert np.array_equal(host8(Q8), Qr) and np.array_equal(SF.cpu().numpy(), chunked_mx(Er, N)), (M, N)
        # 4-bit block-scaled
        gs = 8.0 / 2688.0
        Q4 = torch.full((M, N // 2), 0x55, dtype=torch.uint8, device="cuda")
        SF4 = torch.full((kx.kx_nvfp4_scale_bytes(M, N),), 0xEE, dtype=torch.uint8, device="cuda")
        kx.kx_rmsnorm_quantize_nvfp4(Hd, gd, 1e-6, gs, Q4, SF4)
        Qr, Sr = oracle.quantize_rows_nvfp4(z_bits, gs)
        assert np.array_equal(Q4.cpu().numpy(), Qr) and np.array_equal(SF4.cpu().numpy(), chunked_nv(Sr, N)), (M, N)
        code, detail = kx.kx_last_device_status()
        assert code == kx.KX_OK


@pytest.mark.parametrize("M,N", [(4700, 14336), (6000, 11264), (7000, 9728), (4200, 16384)])
def test_plain_code_books_of_long_rows_in_large_matrices(M, N):
    """From 64 Mi elements on, the plain code books of rows up to 16384 elements run in the short-row kernel with
    five to eight vectors per thread (rows that fill their threads exactly and rows that do not): every format,
    bit for bit."""
    assert M * N >= 64 << 20
    H = inputs.normal_bf16(8100 + N, "R", (M, N), 1.7)
    Hd = kt.to_dev(H)
    Q = torch.full((M, N), 77, dtype=torch.int8, device="cuda")
    S = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
    kx.kx_quantize_rows_int8(Hd, Q, S)
    Qr, Sr = oracle.quantize_rows(H)
    assert np.array_equal(S.cpu().numpy(), Sr) and np.array_equal(Q.cpu().numpy(), Qr)
    del Q
    Q8 = torch.zeros((M, N), dtype=torch.uint8, device="cuda").view(F8)
    kx.kx_quantize_rows_fp8(Hd, Q8, S)
    Qr, Sr = oracle.quantize_rows_fp8(H)
    assert np.array_equal(host8(Q8), Qr) and np.array_equal(S.cpu().numpy(), Sr)
    SF = torch.full((kx.kx_mx_scale_bytes(M, N),), 0xEE, dtype=torch.uint8, device="cuda")
    kx.kx_quantize_rows_mxfp8(Hd, Q8, SF)
    Qr, Er = oracle.quantize_rows_mx(H)
    assert np.array_equal(host8(Q8), Qr) and np.array_equal(SF.cpu().numpy(), chunked_mx(Er, N))
    del Q8
    gs = 8.0 / 2688.0
    Q4 = torch.full((M, N // 2), 0x55, dtype=torch.uint8, device="cuda")
    SF4 = torch.full((kx.kx_nvfp4_scale_bytes(M, N),), 0xEE, dtype=torch.uint8, device="cuda")
    kx.kx_quantize_rows_nvfp4(Hd, gs, Q4, SF4)
    Qr, Sr = oracle.quantize_rows_nvfp4(H, gs)
    assert np.array_equal(Q4.cpu().numpy(), Qr) and np.array_equal(SF4.cpu().numpy(), chunked_nv(Sr, N))
    assert kx.kx_last_device_status()[0] == kx.KX_OK
