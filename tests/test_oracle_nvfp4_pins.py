"""Pins for the oracle's 4-bit block-scaled functions: the element format against its definition and
a brute-force nearest search in exact rationals, the code book against closed forms, invariants and a
step-by-step exact recomputation, the projection against the (separately pinned) BF16 oracle on data
both represent exactly."""
from fractions import Fraction
import math

import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import inputs
from test_oracle_pins import bits
from test_oracle_fp8_pins import exact_value, f64

MAGS = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]


def e2m1_exact(c):
    """E2M1 from its definition: sign, two exponent bits (bias 1), one mantissa bit."""
    s, e, m = (c >> 3) & 1, (c >> 1) & 3, c & 1
    v = Fraction(m, 2) if e == 0 else (1 + Fraction(m, 2)) * Fraction(2) ** (e - 1)
    return -v if s else v


def test_e2m1_decode_is_the_format_definition():
    d = oracle.e2m1_decode(np.arange(16, dtype=np.uint8))
    for c in range(16):
        assert Fraction(float(d[c])) == e2m1_exact(c)
    assert [e2m1_exact(c) for c in range(8)] == MAGS
    assert math.copysign(1.0, d[8]) == -1.0
    assert np.array_equal(oracle.e2m1_decode(np.arange(16, 32, dtype=np.uint8)), d)      # only the low nibble counts


def test_e2m1_encode_nearest_ties_saturation():
    assert np.array_equal(oracle.e2m1_encode(np.float32([float(m) for m in MAGS])), np.arange(8))
    assert np.array_equal(oracle.e2m1_encode(np.float32([-float(m) for m in MAGS])), np.arange(8) | 8)
    mids = np.float32([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    assert oracle.e2m1_encode(mids).tolist() == [0, 2, 2, 4, 4, 6, 6]                    # ties to the even code
    assert oracle.e2m1_encode(np.nextafter(mids, np.float32(np.inf))).tolist() == [1, 2, 3, 4, 5, 6, 7]
    assert oracle.e2m1_encode(np.nextafter(mids, np.float32(0))).tolist() == [0, 1, 2, 3, 4, 5, 6]
    assert oracle.e2m1_encode(np.float32([6.0, 6.5, 1e30, np.inf, -7.0])).tolist() == [7, 7, 7, 7, 15]
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(3000) * 2.5).astype(np.float32)
    got = oracle.e2m1_encode(x)
    for xi, ci in zip(x[::7], got[::7]):
        t = abs(Fraction(float(xi)))
        best = min(abs(m - t) for m in MAGS)
        assert abs(MAGS[int(ci) & 7] - t) == best or t >= 6
        assert (int(ci) >> 3) == (1 if xi < 0 else 0)


def unpack(Q):
    out = np.empty((Q.shape[0], Q.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = Q & 15
    out[:, 1::2] = Q >> 4
    return out


def test_nvfp4_code_book_closed_forms():
    """gs = 1, block = the eight magnitudes (and negatives) times an E4M3-representable scale c: max = 6 c,
    s = e4m3(c) exactly, reciprocal exact when c is a power of two -> the codes come back."""
    vals = np.array([float(m) for m in MAGS])
    for c in (2.0 ** -4, 1.0, 8.0):
        Z = bits((np.concatenate([vals, -vals]) * c).reshape(1, 16))
        Q, S = oracle.quantize_rows_nvfp4(Z, 1.0)
        assert S.shape == (1, 1) and oracle.e4m3_decode(S)[0, 0] == c
        assert unpack(Q)[0].tolist() == list(range(8)) + [c | 8 for c in range(8)]
    # the tensor scale divides out: gs = 2^-3 with the same data gives scale byte for 8 c
    Z = bits((np.concatenate([vals, -vals]) * 0.5).reshape(1, 16))
    Q, S = oracle.quantize_rows_nvfp4(Z, 2.0 ** -3)
    assert oracle.e4m3_decode(S)[0, 0] == 4.0 and unpack(Q)[0, :8].tolist() == list(range(8))
    # zero block: scale byte 0, codes 0; a block whose scale underflows E4M3 also gets codes 0
    Z = bits(np.concatenate([np.zeros(16), np.full(16, 2.0 ** -14)]).reshape(1, 32))
    Q, S = oracle.quantize_rows_nvfp4(Z, 1.0)
    assert S.tolist() == [[0, 0]] and not Q.any()
    # low nibble = even k
    z = np.zeros((1, 16)); z[0, 0] = 6.0; z[0, 1] = -3.0
    Q, S = oracle.quantize_rows_nvfp4(bits(z), 1.0)
    assert Q[0, 0] == (7 | (13 << 4))


def test_nvfp4_code_book_step_by_step_and_invariants():
    Z = inputs.normal_bf16(61, "X", (7, 80), 2.0)
    gs = np.float32(0.013)
    Q, S = oracle.quantize_rows_nvfp4(Z, float(gs))
    zf = inputs.bf16_bits_to_f32(Z)
    codes = unpack(Q)
    assert S.shape == (7, 5)
    for r in range(7):
        for j in range(5):
            blk = zf[r, 16 * j:16 * j + 16]
            a = np.float32(np.abs(blk).max())
            t = np.float32(a / np.float32(np.float32(6.0) * gs))                    # binary32 steps, numpy scalars
            # nearest E4M3 value to t in exact arithmetic (ties to even code)
            tq = Fraction(float(t))
            cands = sorted((abs(exact_value(c) - tq), c % 2, c) for c in range(0x7F))
            assert S[r, j] == cands[0][2]
            sd = np.float32(float(exact_value(int(S[r, j]))))
            rcp = np.float32(np.float32(1.0) / np.float32(sd * gs))
            for k in range(16):
                u = Fraction(float(np.float32(blk[k] * rcp)))
                best = min(abs(m - abs(u)) for m in MAGS)
                c = int(codes[r, 16 * j + k])
                assert abs(u) >= 6 or abs(MAGS[c & 7] - abs(u)) == best
    # the largest element of every block lands on a top code (4 or 6): s is within an E4M3 step of max / 6
    dq = oracle.e2m1_decode(codes) * np.repeat(oracle.e4m3_decode(S), 16, axis=1) * float(gs)
    k = np.abs(zf.reshape(7, 5, 16)).argmax(2)
    top = np.abs(oracle.e2m1_decode(codes).reshape(7, 5, 16))[np.arange(7)[:, None], np.arange(5)[None, :], k]
    assert np.isin(top, [4.0, 6.0]).all()
    # error per element: half an E2M1 step of its binade (relative 1/4 at worst above 0.5, absolute 0.25 below), scaled
    step = np.repeat(oracle.e4m3_decode(S), 16, axis=1) * float(gs)
    assert (np.abs(dq - zf) <= np.maximum(0.25 * np.abs(zf) + 1e-9, 0.25 * step) * 1.07).all()
    Qn, Sn = oracle.quantize_rows_nvfp4(Z ^ np.uint16(0x8000), float(gs))
    assert np.array_equal(Qn, Q ^ 0x88) and np.array_equal(Sn, S)
    Q4, S4 = oracle.quantize_rows_nvfp4(bits(zf.astype(np.float64) * 4.0), float(gs) * 4.0)
    assert np.array_equal(Q4, Q) and np.array_equal(S4, S)                          # a power of two moves into gs


def nv_case(M, N, K, seed):
    rng = np.random.default_rng(seed)
    Xq = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    Wq = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    sx = rng.integers(0x28, 0x48, size=(M, (K + 15) // 16), dtype=np.uint8)       # 2^-2 .. 3.5
    sw = rng.integers(0x20, 0x40, size=(N, (K + 15) // 16), dtype=np.uint8)
    return Xq, sx, Wq, sw


def test_nvfp4_projection_equals_bf16_projection():
    """E2M1 (2 significant bits) times E4M3 (4) times a power of two is BF16-exact (8 bits), so the BF16
    oracle must agree; block j covers k in [16 j, 16 j + 16) of its own row; alpha multiplies the GEMM term
    only."""
    M, N, K = 5, 7, 72                                                             # ragged last block (8 elements)
    Xq, sx, Wq, sw = nv_case(M, N, K, 3)
    X = bits(oracle.e2m1_decode(unpack(Xq)) * np.repeat(oracle.e4m3_decode(sx), 16, axis=1)[:, :K])
    W = bits(oracle.e2m1_decode(unpack(Wq)) * np.repeat(oracle.e4m3_decode(sw), 16, axis=1)[:, :K] * 0.25)
    b = inputs.small_int_bf16(3, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(3, "R", (M, N), -8, 8)
    got = oracle.outproj_nvfp4(Xq, sx, Wq, sw, 0.25, b, R)
    want = oracle.outproj(X, W, b, R)
    assert np.max(np.abs(got - want)) <= 1e-12 * np.abs(want).max()
    rows = np.array([4, 0, 0])
    assert np.array_equal(oracle.outproj_nvfp4(Xq, sx, Wq, sw, 0.25, b, R, rows=rows), got[rows])
    xc, wc = unpack(Xq), unpack(Wq)
    for m, n in ((0, 0), (2, 6), (4, 3)):
        v = Fraction(0)
        for k in range(K):
            v += e2m1_exact(int(xc[m, k])) * e2m1_exact(int(wc[n, k])) * exact_value(int(sx[m, k // 16])) * exact_value(int(sw[n, k // 16]))
        assert oracle.outproj_nvfp4(Xq, sx, Wq, sw, 1.0)[m, n] == pytest.approx(float(v), rel=1e-14, abs=1e-300)
    y1 = oracle.outproj_nvfp4(Xq, sx, Wq, sw, 1.0)
    assert np.allclose(oracle.outproj_nvfp4(Xq, sx, Wq, sw, 3.0, b, R) - oracle.outproj_nvfp4(Xq, sx, Wq, sw, 0.0, b, R), 3.0 * y1, rtol=1e-12)
    # doubling one scale byte's value (exponent field + 1) doubles exactly that block's contribution to that row
    sx2 = sx.copy()
    sx2[1, 2] += 8
    d = oracle.outproj_nvfp4(Xq, sx2, Wq, sw, 1.0) - y1
    assert not d[[0, 2, 3, 4]].any()
    Xb = Xq.copy()
    Xb[:, :16] = 0
    Xb[:, 24:] = 0
    assert np.allclose(d[1], oracle.outproj_nvfp4(Xb, sx, Wq, sw, 1.0)[1], rtol=1e-12, atol=0)


def test_nvfp4_swiglu_equals_bf16_swiglu():
    M, I, K = 5, 9, 48
    Xq, sx, Wgq, sg = nv_case(M, I, K, 8)
    _, _, Wuq, su = nv_case(M, I, K, 9)
    sx[:] = 0x28                                                                   # 0.25
    X = bits(oracle.e2m1_decode(unpack(Xq)) * np.repeat(oracle.e4m3_decode(sx), 16, axis=1)[:, :K] * 0.5)
    Wg = bits(oracle.e2m1_decode(unpack(Wgq)) * np.repeat(oracle.e4m3_decode(sg), 16, axis=1)[:, :K] * 0.25)
    Wu = bits(oracle.e2m1_decode(unpack(Wuq)) * np.repeat(oracle.e4m3_decode(su), 16, axis=1)[:, :K])
    z = oracle.swiglu_nvfp4(Xq, sx, Wgq, sg, Wuq, su, 0.125, 0.5)
    zw, g, u = oracle.swiglu(X, Wg, Wu, want_parts=True)
    assert np.max(np.abs(z - zw)) <= 1e-13 * max(1.0, np.abs(zw).max())
    assert np.abs(g).max() > 0.3
    assert not np.allclose(oracle.swiglu_nvfp4(Xq, sx, Wgq, sg, Wuq, su, 0.5, 0.125), z)   # the two alphas are not interchangeable
    rows = np.array([4, 1])
    assert np.array_equal(oracle.swiglu_nvfp4(Xq, sx, Wgq, sg, Wuq, su, 0.125, 0.5, rows=rows), z[rows])
