"""Pins for the oracle's block-scaled FP8 functions: the scale byte against its definition and a
library conversion, the per-block code book against exact-rational brute force from the format's
definition and against closed forms, and the block-scaled projection against the (separately pinned)
BF16 oracle on data both represent exactly."""
from fractions import Fraction
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import inputs
from test_oracle_pins import bits
from test_oracle_fp8_pins import exact_value, f64


def test_e8m0_decode_is_the_format_definition():
    d = oracle.e8m0_decode(np.arange(256, dtype=np.uint8))
    for e in range(255):
        assert Fraction(float(d[e])) == Fraction(2) ** (e - 127)
    assert math.isnan(d[255])
    assert d[127] == 1.0 and d[0] == 2.0 ** -127 and d[254] == 2.0 ** 127
    if hasattr(torch, "float8_e8m0fnu"):
        lib = torch.arange(255, dtype=torch.uint8).view(torch.float8_e8m0fnu).to(torch.float64).numpy()
        assert np.array_equal(lib, d[:255])


GRID = sorted((exact_value(c), c) for c in range(0x7F))      # non-negative finite codes, by value


def brute_block(vals):
    """One block from the definition, in exact rationals: the scale is the power of two X with
    256 X <= max|v| < 512 X (clamped to the byte range), each element is the grid point nearest to
    v / X (ties to the even code, values above 448 saturate)."""
    a = max(abs(Fraction(float(v))) for v in vals)
    if a == 0:
        e = 127
    else:
        se = -300
        while Fraction(2) ** (se + 1) <= a:
            se += 1                                          # 2^se <= a < 2^(se+1)
        e = min(max(se - 8 + 127, 0), 254)
    X = Fraction(2) ** (e - 127)
    codes = []
    for v in vals:
        t = Fraction(float(v)) / X
        at = abs(t)
        if at >= 448:
            c = 0x7E
        else:
            best = min(abs(g - at) for g, _ in GRID)
            cands = [c for g, c in GRID if abs(g - at) == best]
            c = cands[0] if len(cands) == 1 else [c for c in cands if c % 2 == 0][0]
        codes.append(c | (0x80 if (v < 0 or (v == 0 and math.copysign(1.0, v) < 0)) else 0))
    return e, codes


def test_mx_code_book_against_brute_force():
    rng = np.random.default_rng(11)
    rows = []
    for s in (1e-3, 1.0, 37.0, 2.0 ** -120, 2.0 ** 100):
        rows.append(rng.standard_normal(96) * s)
    rows.append(np.concatenate([rng.standard_normal(32) * 1e-2, rng.standard_normal(32) * 50.0, np.zeros(32)]))
    Zf = np.stack(rows)
    Z = bits(Zf)
    zf = f64(Z)
    Q, E = oracle.quantize_rows_mx(Z)
    assert Q.shape == (6, 96) and E.shape == (6, 3) and Q.dtype == np.uint8 and E.dtype == np.uint8
    for r in range(6):
        for j in range(3):
            e, codes = brute_block(zf[r, 32 * j:32 * j + 32])
            assert E[r, j] == e, (r, j)
            assert Q[r, 32 * j:32 * j + 32].tolist() == codes, (r, j)
    assert E[5, 2] == 127 and not Q[5, 64:].any()            # zero block: scale 1, codes 0
    assert len({int(E[5, 0]), int(E[5, 1]), int(E[5, 2])}) == 3   # blocks of one row scale independently


def test_mx_code_book_closed_forms():
    """Block = E4M3 values times 2^t with the largest magnitude in [256, 512) 2^t: the scale is 2^t and
    the codes come back; a power-of-two maximum 2^p gives byte p - 8 + 127 and code 0x78 (= 256);
    values in (448, 512) X saturate to 448."""
    vals = oracle.e4m3_decode(np.arange(0x5F, 0x7F, dtype=np.uint8))     # 32 codes, max 448
    for t in (-20, 0, 9):
        Z = bits((np.concatenate([vals, -vals]) * 2.0 ** t).reshape(1, 64))
        Q, E = oracle.quantize_rows_mx(Z)
        assert E.tolist() == [[127 + t, 127 + t]]
        assert np.array_equal(Q[0, :32], np.arange(0x5F, 0x7F)) and np.array_equal(Q[0, 32:], np.arange(0x5F, 0x7F) | 0x80)
    for p in (-30, 0, 8, 77):
        z = np.zeros((1, 32))
        z[0, 5] = -(2.0 ** p)
        z[0, 6] = 2.0 ** (p - 3)
        Q, E = oracle.quantize_rows_mx(bits(z))
        assert E[0, 0] == p - 8 + 127 and Q[0, 5] == 0xF8 and Q[0, 6] == 0x60
    z = np.zeros((1, 32))
    z[0, 0], z[0, 1], z[0, 2] = 1.96875, 1.875, 1.75                     # X = 2^-8: 504, 480, 448
    Q, E = oracle.quantize_rows_mx(bits(z))
    assert E[0, 0] == 119 and Q[0, :3].tolist() == [0x7E, 0x7E, 0x7E]
    # smallest scale byte: maxima below 2^-119 keep byte 0
    z = np.zeros((1, 32))
    z[0, 0] = 2.0 ** -125
    Q, E = oracle.quantize_rows_mx(bits(z))
    assert E[0, 0] == 0 and Q[0, 0] == oracle.e4m3_encode(np.float32([4.0]))[0]


def test_mx_code_book_invariants():
    Z = inputs.normal_bf16(41, "X", (9, 160), 3.0)
    Q, E = oracle.quantize_rows_mx(Z)
    zf = f64(Z)
    dq = oracle.e4m3_decode(Q) * np.repeat(oracle.e8m0_decode(E), 32, axis=1)
    X = np.repeat(oracle.e8m0_decode(E), 32, axis=1)
    sat = np.abs(zf) > 448 * X
    assert (np.abs(dq - zf)[~sat] <= (np.abs(zf) * 2.0 ** -4 + X * 2.0 ** -10)[~sat]).all()
    assert np.array_equal(np.abs(dq)[sat], (448 * X)[sat])
    a = np.abs(zf).reshape(9, 5, 32).max(2)
    x5 = oracle.e8m0_decode(E)
    assert (256 * x5 <= a).all() and (a < 512 * x5).all()
    Qn, En = oracle.quantize_rows_mx(Z ^ np.uint16(0x8000))
    assert np.array_equal(Qn, Q ^ 0x80) and np.array_equal(En, E)
    Q8, E8 = oracle.quantize_rows_mx(bits(zf * 8.0))
    assert np.array_equal(Q8, Q) and np.array_equal(E8, E + 3)
    # a ragged last block (cols not a multiple of 32) is a block of its own
    Qr, Er = oracle.quantize_rows_mx(np.ascontiguousarray(Z[:, :150]))
    assert Er.shape == (9, 5) and np.array_equal(Er[:, :4], E[:, :4]) and np.array_equal(Qr[:, :128], Q[:, :128])


def mx_case(M, N, K, seed):
    rng = np.random.default_rng(seed)
    nb = (K + 31) // 32
    Xq = (rng.integers(0, 0x40, size=(M, K), dtype=np.uint8) | (rng.integers(0, 2, size=(M, K), dtype=np.uint8) << 7))
    Wq = (rng.integers(0, 0x40, size=(N, K), dtype=np.uint8) | (rng.integers(0, 2, size=(N, K), dtype=np.uint8) << 7))
    ex = rng.integers(120, 131, size=(M, nb), dtype=np.uint8)
    ew = rng.integers(117, 126, size=(N, nb), dtype=np.uint8)
    return Xq, ex, Wq, ew


def test_mx_projection_equals_bf16_projection():
    """E4M3 values times power-of-two block scales are BF16-exact, so the BF16 oracle must agree; the
    scale of block j covers k in [32 j, 32 j + 32) of its own row only."""
    M, N, K = 5, 7, 100                                       # ragged last block (4 elements)
    Xq, ex, Wq, ew = mx_case(M, N, K, 3)
    X = bits(oracle.e4m3_decode(Xq) * np.repeat(oracle.e8m0_decode(ex), 32, axis=1)[:, :K])
    W = bits(oracle.e4m3_decode(Wq) * np.repeat(oracle.e8m0_decode(ew), 32, axis=1)[:, :K])
    b = inputs.small_int_bf16(3, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(3, "R", (M, N), -8, 8)
    got = oracle.outproj_mx(Xq, ex, Wq, ew, b, R)
    want = oracle.outproj(X, W, b, R)
    assert np.max(np.abs(got - want)) <= 1e-12 * np.abs(want).max()
    rows = np.array([4, 0, 0])
    assert np.array_equal(oracle.outproj_mx(Xq, ex, Wq, ew, b, R, rows=rows), got[rows])
    for m, n in ((0, 0), (2, 6), (4, 3)):
        v = Fraction(0)
        for k in range(K):
            v += (exact_value(int(Xq[m, k])) * exact_value(int(Wq[n, k]))
                  * Fraction(2) ** (int(ex[m, k // 32]) - 127) * Fraction(2) ** (int(ew[n, k // 32]) - 127))
        assert oracle.outproj_mx(Xq, ex, Wq, ew)[m, n] == pytest.approx(float(v), rel=1e-14, abs=1e-300)
    # bumping one scale byte of row m doubles exactly that block's contribution to row m
    ex2 = ex.copy()
    ex2[1, 2] += 1
    d = oracle.outproj_mx(Xq, ex2, Wq, ew) - oracle.outproj_mx(Xq, ex, Wq, ew)
    assert not d[[0, 2, 3, 4]].any()
    Xb = Xq.copy()
    Xb[:, :64] = 0
    Xb[:, 96:] = 0
    assert np.allclose(d[1], oracle.outproj_mx(Xb, ex, Wq, ew)[1], rtol=1e-12, atol=0)
    # NaN scale byte poisons exactly its row
    ex3 = ex.copy()
    ex3[3, 0] = 0xFF
    y = oracle.outproj_mx(Xq, ex3, Wq, ew)
    assert np.isnan(y[3]).all() and not np.isnan(y[[0, 1, 2, 4]]).any()


def test_mx_swiglu_equals_bf16_swiglu():
    """On operands the BF16 format represents exactly, the (separately pinned) BF16 SwiGLU oracle must agree;
    gate and up are not interchangeable."""
    M, I, K = 5, 9, 96
    Xq, ex, Wgq, eg = mx_case(M, I, K, 8)
    _, _, Wuq, eu = mx_case(M, I, K, 9)
    Xq &= 0xB7                      # |x| < 1
    ex[:] = 127
    X = bits(oracle.e4m3_decode(Xq) * np.repeat(oracle.e8m0_decode(ex), 32, axis=1))
    Wg = bits(oracle.e4m3_decode(Wgq) * np.repeat(oracle.e8m0_decode(eg), 32, axis=1))
    Wu = bits(oracle.e4m3_decode(Wuq) * np.repeat(oracle.e8m0_decode(eu), 32, axis=1))
    z = oracle.swiglu_mx(Xq, ex, Wgq, eg, Wuq, eu)
    zw, g, u = oracle.swiglu(X, Wg, Wu, want_parts=True)
    assert np.max(np.abs(z - zw)) <= 1e-13 * max(1.0, np.abs(zw).max())
    assert np.abs(g).max() > 0.3
    assert not np.allclose(oracle.swiglu_mx(Xq, ex, Wuq, eu, Wgq, eg), z)
    rows = np.array([4, 1])
    assert np.array_equal(oracle.swiglu_mx(Xq, ex, Wgq, eg, Wuq, eu, rows=rows), z[rows])
