"""Pins for the oracle's INT8 branch: the per-row code book against exact rational
arithmetic, closed forms and the defining properties of round-to-nearest; the INT8
gate/up + SwiGLU and the INT8 projection against the (separately pinned) BF16 oracle
functions on data where both are exact, and against brute force on tiny cases."""
from fractions import Fraction
import math

import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import inputs
from test_oracle_pins import bits


def f64(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


# ------------------------------------------------------------------ quantize_rows
def test_codes_on_an_exact_grid():
    """Row = j * 2^e for j in -127..127 (all BF16-exact): max|z| = 127 * 2^e, so scale = 2^e and
    127 / max|z| = 2^-e exactly, every product is the integer j, and the codes are j."""
    for e in (-9, 0, 5):
        j = np.arange(-127, 128, dtype=np.float64)
        Z = bits((j * 2.0 ** e).reshape(1, -1))
        Q, S = oracle.quantize_rows(Z)
        assert Q.dtype == np.int8 and S.dtype == np.float32
        assert np.array_equal(Q[0], j.astype(np.int8))
        assert S[0] == np.float32(2.0 ** e)


def test_ties_go_to_the_even_code():
    """With 127 * 2^e in the row the products (j + 1/2) are exact: round half to even."""
    vals = np.array([127.0, 0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, 62.5, 63.5, -63.5])
    want = np.array([127, 0, 2, 2, 4, 0, -2, -2, 62, 64, -64], dtype=np.int8)
    Q, S = oracle.quantize_rows(bits(vals.reshape(1, -1) * 0.25))
    assert np.array_equal(Q[0], want) and S[0] == np.float32(0.25)


def test_zero_row_and_single_value_rows():
    Z = bits(np.array([[0.0, -0.0, 0.0], [0.0, 0.0, -3.0], [7.0, 7.0, 7.0]]))
    Q, S = oracle.quantize_rows(Z)
    assert np.array_equal(Q[0], [0, 0, 0]) and S[0] == np.float32(1.0)
    assert np.array_equal(Q[1], [0, 0, -127]) and S[1] == np.float32(3.0) / np.float32(127.0)
    assert np.array_equal(Q[2], [127, 127, 127])
    Q0, S0 = oracle.quantize_rows(np.zeros((0, 8), dtype=np.uint16))
    assert Q0.shape == (0, 8) and S0.shape == (0,)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_nearest_code_in_exact_arithmetic(seed):
    """Against exact rationals: t = 127 z / max|z|.  The code is one of the two integers around t,
    and the nearest one whenever t is further than 2^-15 |t| from a tie (binary32 rounding of the
    reciprocal and of the product moves t by at most about 2^-23 relative each)."""
    Z = inputs.normal_bf16(seed, "X", (6, 257), 3.0)
    Q, S = oracle.quantize_rows(Z)
    zf = f64(Z)
    for r in range(Z.shape[0]):
        a = Fraction(float(np.abs(zf[r]).max()))
        assert S[r] == np.float32(np.float32(float(a)) / np.float32(127.0))
        for j in range(Z.shape[1]):
            t = Fraction(float(zf[r, j])) * 127 / a
            q = int(Q[r, j])
            assert math.floor(t) <= q <= math.ceil(t), (r, j, float(t), q)
            frac = t - math.floor(t)
            if abs(frac - Fraction(1, 2)) > abs(t) * Fraction(1, 2 ** 15) + Fraction(1, 2 ** 30):
                assert q == math.floor(t + Fraction(1, 2)), (r, j, float(t), q)


def test_defining_properties():
    """Every non-zero row reaches +-127 exactly at its largest element; codes are monotone in z;
    |z - q * scale| <= scale / 2 (+ rounding slack); negating a row negates its codes; scaling a
    row by a power of two scales the scale and keeps the codes; rows are independent."""
    Z = inputs.normal_bf16(11, "X", (40, 300), 1.0)
    zf = f64(Z)
    Q, S = oracle.quantize_rows(Z)
    for r in range(Z.shape[0]):
        k = int(np.argmax(np.abs(zf[r])))
        assert abs(int(Q[r, k])) == 127 and np.sign(Q[r, k]) == np.sign(zf[r, k])
        assert np.abs(Q[r].astype(np.int32)).max() == 127
        order = np.argsort(zf[r], kind="stable")
        assert (np.diff(Q[r, order].astype(np.int32)) >= 0).all()
        err = np.abs(zf[r] - Q[r].astype(np.float64) * float(S[r]))
        assert err.max() <= 0.5 * float(S[r]) * (1 + 1e-5)
    Qn, Sn = oracle.quantize_rows(Z ^ np.uint16(0x8000))
    assert np.array_equal(Qn, -Q) and np.array_equal(Sn, S)
    Q4, S4 = oracle.quantize_rows(bits(zf * 16.0))
    assert np.array_equal(Q4, Q) and np.array_equal(S4, S * np.float32(16.0))
    Qs, Ss = oracle.quantize_rows(Z[7:9])
    assert np.array_equal(Qs, Q[7:9]) and np.array_equal(Ss, S[7:9])


# ------------------------------------------------------------------ INT8 GEMMs
def int8_case(M, N, K, seed=5):
    rng = np.random.default_rng(seed)
    Xq = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    Wq = rng.integers(-127, 128, size=(N, K), dtype=np.int8)
    return Xq, Wq


def pow2_scales(n, seed):
    rng = np.random.default_rng(seed)
    return (2.0 ** rng.integers(-9, -3, size=n)).astype(np.float32)


def test_int8_projection_equals_bf16_projection_on_power_of_two_scales():
    """Codes (|q| <= 127) and power-of-two scales are BF16-exact, so X = Xq * sx and W = Wq * sw
    are exact BF16 matrices and the (separately pinned) BF16 projection must agree: the integer
    sum, both scale factors, bias and residual all show up."""
    M, N, K = 7, 12, 45
    Xq, Wq = int8_case(M, N, K)
    sx, sw = pow2_scales(M, 1), pow2_scales(N, 2)
    X = bits(Xq.astype(np.float64) * sx[:, None].astype(np.float64))
    W = bits(Wq.astype(np.float64) * sw[:, None].astype(np.float64))
    b = inputs.small_int_bf16(3, "bias", (N,), -4, 4)
    R = inputs.small_int_bf16(3, "R", (M, N), -8, 8)
    got = oracle.outproj_int8(Xq, sx, Wq, sw, b, R)
    want = oracle.outproj(X, W, b, R)
    assert np.max(np.abs(got - want)) <= 1e-12 * np.abs(want).max()
    assert np.array_equal(oracle.outproj_int8(Xq, sx, Wq, sw), oracle.outproj(X, W))  # both exact
    rows = np.array([6, 0, 2, 2])
    assert np.array_equal(oracle.outproj_int8(Xq, sx, Wq, sw, b, R, rows=rows), got[rows])


def test_int8_projection_brute_force_and_scale_axes():
    M, N, K = 3, 4, 9
    Xq, Wq = int8_case(M, N, K, seed=8)
    sx = np.array([0.013, 0.5, 3.0], dtype=np.float32)
    sw = np.array([1.0, 0.37, 0.002, 11.0], dtype=np.float32)
    got = oracle.outproj_int8(Xq, sx, Wq, sw)
    for m in range(M):
        for n in range(N):
            acc = sum(int(Xq[m, k]) * int(Wq[n, k]) for k in range(K))
            want = Fraction(acc) * Fraction(float(sx[m])) * Fraction(float(sw[n]))
            assert got[m, n] == pytest.approx(float(want), rel=1e-15, abs=1e-300)
    # swapping the scale vectors' roles must change the result (row scale is per m, column per n)
    assert not np.allclose(got, oracle.outproj_int8(Xq, np.ones(M, np.float32), Wq, sw))
    assert np.allclose(got, oracle.outproj_int8(Xq, np.ones(M, np.float32), Wq, sw) * sx[:, None].astype(np.float64))


def test_int8_swiglu_equals_bf16_swiglu_on_power_of_two_scales():
    M, I, K = 6, 10, 33
    Xq, Wgq = int8_case(M, I, K, seed=9)
    _, Wuq = int8_case(M, I, K, seed=10)
    sx, sg, su = pow2_scales(M, 4), pow2_scales(I, 5), pow2_scales(I, 6)
    # keep the pre-activations moderate so that silu is not saturated
    sx = (sx / 64).astype(np.float32)
    X = bits(Xq.astype(np.float64) * sx[:, None])
    Wg = bits(Wgq.astype(np.float64) * sg[:, None])
    Wu = bits(Wuq.astype(np.float64) * su[:, None])
    z, ga, ua = oracle.swiglu_int8(Xq, sx, Wgq, sg, Wuq, su, want_acc=True)
    zw, g, u = oracle.swiglu(X, Wg, Wu, want_parts=True)
    assert np.array_equal(ga, Xq.astype(np.int64) @ Wgq.astype(np.int64).T)
    assert np.array_equal(ua, Xq.astype(np.int64) @ Wuq.astype(np.int64).T)
    assert np.array_equal(ga * sx[:, None].astype(np.float64) * sg[None, :].astype(np.float64), g)
    assert np.max(np.abs(z - zw)) <= 1e-13 * max(1.0, np.abs(zw).max())
    assert np.abs(g).max() > 0.5 and np.abs(g).min() < 50      # silu exercised off its asymptotes
    # the gate goes through silu, the up factor multiplies
    sw = oracle.swiglu_int8(Xq, sx, Wuq, su, Wgq, sg)
    assert not np.allclose(sw, z)
    rows = np.array([5, 1, 1])
    assert np.array_equal(oracle.swiglu_int8(Xq, sx, Wgq, sg, Wuq, su, rows=rows), z[rows])


def test_int8_swiglu_brute_force():
    M, I, K = 2, 3, 5
    Xq, Wgq = int8_case(M, I, K, seed=12)
    _, Wuq = int8_case(M, I, K, seed=13)
    sx = np.array([0.01, 0.002], dtype=np.float32)
    sg = np.array([0.02, 0.005, 0.01], dtype=np.float32)
    su = np.array([0.5, 0.25, 3.0], dtype=np.float32)
    z = oracle.swiglu_int8(Xq, sx, Wgq, sg, Wuq, su)
    for m in range(M):
        for i in range(I):
            g = sum(int(Xq[m, k]) * int(Wgq[i, k]) for k in range(K)) * float(sx[m]) * float(sg[i])
            u = sum(int(Xq[m, k]) * int(Wuq[i, k]) for k in range(K)) * float(sx[m]) * float(su[i])
            assert z[m, i] == pytest.approx(g / (1.0 + math.exp(-g)) * u, rel=1e-14)


def test_quantise_then_project_tracks_the_bf16_projection():
    """End to end: quantising X and W with the code book and projecting on the codes stays within
    the quantisation error bound of the BF16 projection: |y8 - y| <= sum_k (|x| sw/2 + |w| sx/2 +
    sx sw / 4) per element, a bound that holds for round-to-nearest codes and fails for a wrong
    scale, a transposed scale or truncation."""
    M, N, K = 9, 13, 200
    X = inputs.normal_bf16(21, "X", (M, K), 1.0)
    W = inputs.normal_bf16(21, "W", (N, K), 0.07)
    Xq, sx = oracle.quantize_rows(X)
    Wq, sw = oracle.quantize_rows(W)
    y8 = oracle.outproj_int8(Xq, sx, Wq, sw)
    y = oracle.outproj(X, W)
    ax, aw = np.abs(f64(X)), np.abs(f64(W))
    bound = (ax.sum(1)[:, None] * sw[None, :] / 2 + aw.sum(1)[None, :] * sx[:, None] / 2
             + K * sx[:, None] * sw[None, :] / 4) * (1 + 1e-5)
    assert (np.abs(y8 - y) <= bound).all()
    assert np.abs(y8 - y).max() > 0           # it is a different computation
    rms = np.sqrt(np.mean((y8 - y) ** 2)) / np.sqrt(np.mean(y ** 2))
    assert rms < 0.02


def test_hand_computed_code_book_fixture():
    """tests/golden/quantize_rows_8bit.txt: rows whose scale is a power of two, codes worked out by hand
    (ties to even for INT8; E4M3 bit patterns from the format definition)."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "quantize_rows_8bit.txt")
    fmt, scale, z = None, None, None
    checked = 0
    for line in open(path):
        line = line.split("#")[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] in ("int8", "fp8"):
            fmt = tok[0]
        elif tok[0] == "scale":
            scale = float(tok[1])
        elif tok[0] == "z":
            z = np.array([float(t) for t in tok[1:]])
        elif tok[0] == "q":
            want = np.array([int(t, 0) for t in tok[1:]])
            Z = bits(z.reshape(1, -1))
            assert np.array_equal(inputs.bf16_bits_to_f32(Z)[0].astype(np.float64), z)      # fixture is BF16-exact
            if fmt == "int8":
                Q, S = oracle.quantize_rows(Z)
                assert np.array_equal(Q[0].astype(np.int64), want), (Q[0], want)
            else:
                Q, S = oracle.quantize_rows_fp8(Z)
                assert np.array_equal(Q[0].astype(np.int64), want), ([hex(v) for v in Q[0]], want)
            assert S[0] == np.float32(scale)
            checked += 1
    assert checked == 3
