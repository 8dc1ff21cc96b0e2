"""Pins for the oracle's FP8 (E4M3) functions: the format itself against its definition and a
library conversion, the rounding against exact rationals, the per-row code book against closed
forms, and the FP8 GEMMs against the (separately pinned) BF16 oracle functions on data both
represent exactly."""
from fractions import Fraction
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import inputs
from test_oracle_pins import bits


ALL = np.arange(256, dtype=np.uint8)


def f64(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def exact_value(code: int):
    """E4M3 from its definition, field by field, as an exact rational (None for NaN)."""
    s, e, m = code >> 7, (code >> 3) & 15, code & 7
    if e == 15 and m == 7:
        return None
    v = Fraction(m, 8) * Fraction(1, 64) if e == 0 else (1 + Fraction(m, 8)) * Fraction(2) ** (e - 7)
    return -v if s else v


def test_decode_is_the_format_definition():
    d = oracle.e4m3_decode(ALL)
    for c in range(256):
        v = exact_value(c)
        if v is None:
            assert math.isnan(d[c])
        else:
            assert Fraction(float(d[c])) == v
    assert d[0x7E] == 448.0 and d[0x08] == 2.0 ** -6 and d[0x01] == 2.0 ** -9 and d[0x38] == 1.0
    assert math.copysign(1.0, d[0x80]) == -1.0 and d[0x80] == 0.0
    lib = torch.from_numpy(ALL.copy()).view(torch.float8_e4m3fn).float().numpy()
    assert np.array_equal(np.isnan(d), np.isnan(lib)) and np.array_equal(d[~np.isnan(d)], lib[~np.isnan(lib)])


def test_encode_round_trip_ties_saturation():
    d = oracle.e4m3_decode(ALL)
    fin = ~np.isnan(d)
    assert np.array_equal(oracle.e4m3_encode(d[fin].astype(np.float32)), ALL[fin])
    # midpoints between neighbouring positive codes go to the even code
    pos = np.arange(0, 0x7E, dtype=np.uint8)
    mid = ((d[pos] + d[pos + 1]) / 2).astype(np.float32)            # exact in binary32
    got = oracle.e4m3_encode(mid)
    want = np.where(pos % 2 == 0, pos, pos + 1).astype(np.uint8)
    assert np.array_equal(got, want)
    assert np.array_equal(oracle.e4m3_encode(-mid), want | 0x80)
    # just off the midpoint: nearest wins
    assert np.array_equal(oracle.e4m3_encode(np.nextafter(mid, np.float32(np.inf))), pos + 1)
    assert np.array_equal(oracle.e4m3_encode(np.nextafter(mid, np.float32(0))), pos)
    # saturation instead of overflow, NaN code for NaN, tiny values flush to zero
    x = np.array([448.0, 449.0, 464.0, 465.0, 1e30, np.inf, -500.0, 2.0 ** -10, 2.0 ** -11, np.nan], np.float32)
    assert oracle.e4m3_encode(x).tolist() == [0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0x00, 0x00, 0x7F]


def test_encode_is_nearest_in_exact_arithmetic_and_matches_library():
    rng = np.random.default_rng(4)
    x = np.concatenate([rng.standard_normal(4000) * s for s in (1e-3, 0.05, 1.0, 30.0, 200.0)]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    got = oracle.e4m3_encode(x)
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(got, lib)
    grid = sorted(exact_value(c) for c in range(0x7F))
    for xi, ci in zip(x[::37], got[::37]):
        v, t = abs(exact_value(int(ci))), abs(Fraction(float(xi)))
        best = min(abs(g - t) for g in grid)
        assert abs(v - t) == best


def test_fp8_code_book():
    """Row = the 127 positive finite code values times 2^e: max = 448 * 2^e, scale = 2^e and 448 / max = 2^-e
    exactly, products are the code values themselves -> the codes come back; zero rows; scale of a
    general row is one binary32 division; every element stays within half a code step."""
    vals = oracle.e4m3_decode(np.arange(1, 0x7F, dtype=np.uint8))
    for e in (-5, 0, 3):
        # BF16 has 8 significand bits: every E4M3 value (4 bits) times 2^e is BF16-exact
        Z = bits(np.concatenate([vals, -vals]).reshape(1, -1) * 2.0 ** e)
        Q, S = oracle.quantize_rows_fp8(Z)
        assert Q.dtype == np.uint8 and S.dtype == np.float32
        assert S[0] == np.float32(2.0 ** e)
        assert np.array_equal(Q[0, :126], np.arange(1, 0x7F)) and np.array_equal(Q[0, 126:], np.arange(1, 0x7F) | 0x80)
    Q, S = oracle.quantize_rows_fp8(bits(np.zeros((2, 16))))
    assert not Q.any() and (S == 1.0).all()
    Z = inputs.normal_bf16(31, "X", (12, 400), 2.0)
    Q, S = oracle.quantize_rows_fp8(Z)
    zf = f64(Z)
    a = np.abs(zf).max(1)
    assert np.array_equal(S, (a.astype(np.float32) / np.float32(448.0)))
    dq = oracle.e4m3_decode(Q) * S[:, None].astype(np.float64)
    # half a step: 2^-4 relative for normal codes (3 mantissa bits), 2^-10 * 448-scale absolute for subnormals
    assert (np.abs(dq - zf) <= np.abs(zf) * 2.0 ** -4 * (1 + 1e-5) + S[:, None] * 2.0 ** -10 * (1 + 1e-5)).all()
    k = np.argmax(np.abs(zf), 1)
    assert (Q[np.arange(12), k] & 0x7F == 0x7E).all()
    Qn, Sn = oracle.quantize_rows_fp8(Z ^ np.uint16(0x8000))
    assert np.array_equal(Qn, Q ^ 0x80) and np.array_equal(Sn, S)
    Q4, S4 = oracle.quantize_rows_fp8(bits(zf * 4.0))
    assert np.array_equal(Q4, Q) and np.array_equal(S4, S * np.float32(4.0))


def fp8_case(M, N, K, seed):
    rng = np.random.default_rng(seed)
    # finite codes only (no 0x7F / 0xFF)
    Xq = rng.integers(0, 0x7F, size=(M, K), dtype=np.uint8) | (rng.integers(0, 2, size=(M, K), dtype=np.uint8) << 7)
    Wq = rng.integers(0, 0x7F, size=(N, K), dtype=np.uint8) | (rng.integers(0, 2, size=(N, K), dtype=np.uint8) << 7)
    return Xq, Wq


def test_fp8_projection_equals_bf16_projection():
    """E4M3 values times power-of-two scales are BF16-exact, so the BF16 oracle must agree."""
    M, N, K = 6, 11, 37
    Xq, Wq = fp8_case(M, N, K, 7)
    Xq &= 0xBF                      # keep |x| < 2 so that products stay moderate
    sx = (2.0 ** np.random.default_rng(1).integers(-4, 2, M)).astype(np.float32)
    sw = (2.0 ** np.random.default_rng(2).integers(-6, -1, N)).astype(np.float32)
    X = bits(oracle.e4m3_decode(Xq) * sx[:, None])
    W = bits(oracle.e4m3_decode(Wq) * sw[:, None])
    b = inputs.small_int_bf16(3, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(3, "R", (M, N), -8, 8)
    got = oracle.outproj_fp8(Xq, sx, Wq, sw, b, R)
    want = oracle.outproj(X, W, b, R)
    assert np.max(np.abs(got - want)) <= 1e-12 * np.abs(want).max()
    rows = np.array([5, 0, 0])
    assert np.array_equal(oracle.outproj_fp8(Xq, sx, Wq, sw, b, R, rows=rows), got[rows])
    # brute force, exact rationals
    for m, n in ((0, 0), (3, 7), (5, 10)):
        acc = sum(exact_value(int(Xq[m, k])) * exact_value(int(Wq[n, k])) for k in range(K))
        v = acc * Fraction(float(sx[m])) * Fraction(float(sw[n]))
        assert oracle.outproj_fp8(Xq, sx, Wq, sw)[m, n] == pytest.approx(float(v), rel=1e-14, abs=1e-300)
    # the row scale belongs to m, the column scale to n
    one = np.ones(M, np.float32)
    assert np.allclose(oracle.outproj_fp8(Xq, one, Wq, sw) * sx[:, None].astype(np.float64), oracle.outproj_fp8(Xq, sx, Wq, sw))


def test_fp8_swiglu_equals_bf16_swiglu():
    M, I, K = 5, 9, 29
    Xq, Wgq = fp8_case(M, I, K, 8)
    _, Wuq = fp8_case(M, I, K, 9)
    Xq &= 0xB7                      # |x| < 1
    Wgq &= 0xBF
    sx = np.full(M, 1.0, np.float32)
    sg = (2.0 ** np.random.default_rng(5).integers(-3, 0, I)).astype(np.float32)
    su = (2.0 ** np.random.default_rng(6).integers(-6, -2, I)).astype(np.float32)
    X = bits(oracle.e4m3_decode(Xq) * sx[:, None])
    Wg = bits(oracle.e4m3_decode(Wgq) * sg[:, None])
    Wu = bits(oracle.e4m3_decode(Wuq) * su[:, None])
    z = oracle.swiglu_fp8(Xq, sx, Wgq, sg, Wuq, su)
    zw, g, u = oracle.swiglu(X, Wg, Wu, want_parts=True)
    assert np.max(np.abs(z - zw)) <= 1e-13 * max(1.0, np.abs(zw).max())
    assert np.abs(g).max() > 0.3
    assert not np.allclose(oracle.swiglu_fp8(Xq, sx, Wuq, su, Wgq, sg), z)     # gate and up are not interchangeable
    rows = np.array([4, 1])
    assert np.array_equal(oracle.swiglu_fp8(Xq, sx, Wgq, sg, Wuq, su, rows=rows), z[rows])
