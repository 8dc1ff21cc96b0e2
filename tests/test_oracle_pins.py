"""Pins for the CPU oracle: everything here checks the oracle against something
other than itself — exact rational brute force, a hand-computed fixture, a
float64 library matmul, closed forms and invariants."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def frac_of_bits(b: int) -> Fraction:
    """Exact value of a finite BF16 bit pattern, decoded field by field."""
    sign = -1 if (b >> 15) & 1 else 1
    e = (b >> 7) & 0xFF
    m = b & 0x7F
    assert e != 0xFF
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(1, 1 << 126)
    mant = Fraction((1 << 7) + m, 1 << 7)
    return sign * mant * (Fraction(2) ** (e - 127))


def brute(X, W, bias, R):
    M, K = X.shape
    N = W.shape[0]
    out = [[Fraction(0)] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            s = Fraction(0)
            for k in range(K):
                s += frac_of_bits(int(X[m, k])) * frac_of_bits(int(W[n, k]))
            if bias is not None:
                s += frac_of_bits(int(bias[n]))
            if R is not None:
                s += frac_of_bits(int(R[m, n]))
            out[m][n] = s
    return out


def bits(a):
    return inputs.f32_to_bf16_bits(np.asarray(a, dtype=np.float32)).reshape(np.shape(a))


# ---------------------------------------------------------------- fixture
def _read_golden(path):
    sec, data = None, {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] in ("M", "N", "K"):
            data[tok[0]] = int(tok[1])
        elif tok[0][0].isalpha():
            sec = tok[0]
            data[sec] = []
        else:
            data[sec].append([float(t) for t in tok])
    return data


def test_hand_computed_fixture():
    g = _read_golden(os.path.join(GOLDEN, "outproj_2x3x2.txt"))
    X, W = bits(g["X"]), bits(g["W"])
    bias, R = bits(g["bias"][0]), bits(g["R"])
    assert X.shape == (g["M"], g["K"]) and W.shape == (g["N"], g["K"])
    ref = oracle.outproj(X, W, bias, R)
    assert np.array_equal(ref, np.array(g["Y"]))
    assert np.array_equal(oracle.outproj(X, W), np.array(g["Y_plain"]))


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (2, 2, 2), (3, 5, 7), (8, 6, 32), (5, 9, 17), (4, 7, 0)])
@pytest.mark.parametrize("has_bias,has_R", [(False, False), (True, False), (False, True), (True, True)])
def test_exact_brute_force_small_ints(M, N, K, has_bias, has_R):
    """Integer-valued inputs: every partial sum is an integer, so the double
    result must equal the exact rational result."""
    X = inputs.small_int_bf16(100 + M, "X", (M, K))
    W = inputs.small_int_bf16(100 + N, "W", (N, K))
    bias = inputs.small_int_bf16(7, "bias", (N,)) if has_bias else None
    R = inputs.small_int_bf16(9, "R", (M, N)) if has_R else None
    ref, absref = oracle.outproj(X, W, bias, R, want_abs=True)
    ex = brute(X, W, bias, R)
    ab = brute(*(None if a is None else (a & np.uint16(0x7FFF)) for a in (X, W, bias, R)))
    for m in range(M):
        for n in range(N):
            assert Fraction(ref[m, n]) == ex[m][n], (m, n)
            assert Fraction(absref[m, n]) == ab[m][n], (m, n)


@pytest.mark.parametrize("M,N,K", [(2, 3, 4), (4, 5, 16), (3, 6, 33)])
def test_brute_force_random_values(M, N, K):
    """Random BF16 values: the double sum may round, but only at the 2^-53 level
    relative to the sum of magnitudes."""
    wl = inputs.Workload("t", M, N, K, 1234, True, True)
    d = inputs.make_inputs(wl, stress=True)
    ref, absref = oracle.outproj(d["X"], d["W"], d["bias"], d["R"], want_abs=True)
    ex = brute(d["X"], d["W"], d["bias"], d["R"])
    for m in range(M):
        for n in range(N):
            err = abs(Fraction(ref[m, n]) - ex[m][n])
            assert err <= Fraction(absref[m, n]) * Fraction(K + 2, 1 << 52), (m, n)


# ---------------------------------------------------------------- library routine
@pytest.mark.parametrize("M,N,K", [(7, 13, 64), (33, 130, 257), (128, 96, 512)])
def test_against_float64_matmul(M, N, K):
    wl = inputs.Workload("t", M, N, K, 77, True, True)
    d = inputs.make_inputs(wl)
    Xd = torch.from_numpy(inputs.bf16_bits_to_f32(d["X"]).astype(np.float64))
    Wd = torch.from_numpy(inputs.bf16_bits_to_f32(d["W"]).astype(np.float64))
    bd = torch.from_numpy(inputs.bf16_bits_to_f32(d["bias"]).astype(np.float64))
    Rd = torch.from_numpy(inputs.bf16_bits_to_f32(d["R"]).astype(np.float64))
    lib = (Xd @ Wd.T + bd + Rd).numpy()
    ref = oracle.outproj(d["X"], d["W"], d["bias"], d["R"])
    assert np.max(np.abs(ref - lib)) <= 1e-12 * max(1.0, np.max(np.abs(lib)))
    # plain GEMM and the bias-only / residual-only forms
    assert np.max(np.abs(oracle.outproj(d["X"], d["W"]) - (Xd @ Wd.T).numpy())) <= 1e-12
    assert np.max(np.abs(oracle.outproj(d["X"], d["W"], d["bias"]) - (Xd @ Wd.T + bd).numpy())) <= 1e-12
    assert np.max(np.abs(oracle.outproj(d["X"], d["W"], None, d["R"]) - (Xd @ Wd.T + Rd).numpy())) <= 1e-12


def test_rows_and_element_modes_agree_with_full():
    wl = inputs.Workload("t", 300, 70, 96, 5, True, True)
    d = inputs.make_inputs(wl)
    full = oracle.outproj(d["X"], d["W"], d["bias"], d["R"])
    rows = inputs.sampled_rows(300)
    assert rows[0] == 0 and rows[-1] == 299 and len(set(rows.tolist())) == len(rows)
    part, _ = oracle.outproj_rows(d["X"], d["W"], d["bias"], d["R"], rows)
    assert np.array_equal(part, full[rows])
    # a permuted, repeated row list
    rr = np.array([299, 5, 5, 0, 128], dtype=np.int64)
    part, _ = oracle.outproj_rows(d["X"], d["W"], d["bias"], d["R"], rr)
    assert np.array_equal(part, full[rr])
    for (m, n) in [(0, 0), (299, 69), (17, 3), (128, 64)]:
        assert oracle.element(d["X"], d["W"], d["bias"], d["R"], m, n) == full[m, n]
    assert oracle.outproj(d["X"], d["W"], d["bias"], d["R"], threads=1).tobytes() == full.tobytes()


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("K", [1, 8, 100, 4096])
def test_constant_operands_closed_form(K):
    M, N = 5, 11
    a, b = 0.5, 4.0
    X = bits(np.full((M, K), a))
    W = bits(np.full((N, K), b))
    bias = inputs.small_int_bf16(1, "bias", (N,))
    R = inputs.small_int_bf16(2, "R", (M, N))
    ref = oracle.outproj(X, W, bias, R)
    want = K * a * b + inputs.bf16_bits_to_f32(bias)[None, :].astype(np.float64) \
        + inputs.bf16_bits_to_f32(R).astype(np.float64)
    assert np.array_equal(ref, want)


def test_one_hot_rows_select_columns_of_W():
    M, N, K = 37, 19, 24
    X = inputs.one_hot_rows_bf16(M, K)
    W = inputs.normal_bf16(3, "W", (N, K), 1.0)
    ref = oracle.outproj(X, W)
    Wf = inputs.bf16_bits_to_f32(W).astype(np.float64)
    for m in range(M):
        assert np.array_equal(ref[m], Wf[:, m % K])


def test_permutation_W_selects_columns_of_X():
    M, N, K = 9, 20, 31
    W, pi = inputs.permutation_matrix_bf16(4, N, K)
    X = inputs.normal_bf16(4, "X", (M, K), 1.0)
    R = inputs.normal_bf16(4, "R", (M, N), 1.0)
    ref = oracle.outproj(X, W, None, R)
    Xf = inputs.bf16_bits_to_f32(X).astype(np.float64)
    Rf = inputs.bf16_bits_to_f32(R).astype(np.float64)
    assert np.array_equal(ref, Xf[:, pi] + Rf)


# ---------------------------------------------------------------- invariants
def test_zero_weight_gives_residual_plus_bias():
    M, N, K = 6, 10, 40
    d = inputs.make_inputs(inputs.Workload("t", M, N, K, 11, True, True))
    W0 = np.zeros((N, K), dtype=np.uint16)
    ref = oracle.outproj(d["X"], W0, d["bias"], d["R"])
    want = inputs.bf16_bits_to_f32(d["R"]).astype(np.float64) \
        + inputs.bf16_bits_to_f32(d["bias"]).astype(np.float64)[None, :]
    assert np.array_equal(ref, want)
    assert np.array_equal(oracle.outproj(d["X"], W0), np.zeros((M, N)))


def test_identity_weight_gives_x_plus_residual_plus_bias():
    M, N = 7, 12
    d = inputs.make_inputs(inputs.Workload("t", M, N, N, 12, True, True), stress=True)
    I = bits(np.eye(N))
    ref = oracle.outproj(d["X"], I, d["bias"], d["R"])
    f = lambda a: inputs.bf16_bits_to_f32(a).astype(np.float64)
    # (x + bias) + R in double: x, bias, R are BF16 so every sum is exact
    assert np.array_equal(ref, f(d["X"]) + f(d["bias"])[None, :] + f(d["R"]))


def test_linearity_in_X():
    M, N, K = 5, 8, 48
    X1 = inputs.small_int_bf16(1, "X", (M, K), -7, 7)
    X2 = inputs.small_int_bf16(2, "X", (M, K), -7, 7)
    W = inputs.small_int_bf16(3, "W", (N, K), -7, 7)
    Xs = bits(inputs.bf16_bits_to_f32(X1) + inputs.bf16_bits_to_f32(X2))
    X3 = bits(3.0 * inputs.bf16_bits_to_f32(X1))
    r1, r2 = oracle.outproj(X1, W), oracle.outproj(X2, W)
    assert np.array_equal(oracle.outproj(Xs, W), r1 + r2)
    assert np.array_equal(oracle.outproj(X3, W), 3.0 * r1)
    # scaling by a power of two is exact for arbitrary values
    Xr = inputs.normal_bf16(5, "X", (M, K), 1.0)
    Wr = inputs.normal_bf16(5, "W", (N, K), 1.0)
    X2r = bits(2.0 * inputs.bf16_bits_to_f32(Xr))
    assert np.array_equal(oracle.outproj(X2r, Wr), 2.0 * oracle.outproj(Xr, Wr))


def test_sum_order_is_increasing_k():
    """Products 1, 2^-53, 2^-53 summed term by term in increasing k give exactly
    1.0 (each tiny addend is a tie that rounds back to the even value 1.0);
    summed in decreasing k they give 1 + 2^-52.  The exact value is 1 + 2^-52."""
    X = bits(np.array([[1.0, 2.0 ** -26, 2.0 ** -26]]))
    W = bits(np.array([[1.0, 2.0 ** -27, 2.0 ** -27]]))
    assert oracle.outproj(X, W)[0, 0] == 1.0
    assert oracle.outproj(X[:, ::-1].copy(), W[:, ::-1].copy())[0, 0] == 1.0 + 2.0 ** -52
    assert brute(X, W, None, None)[0][0] == 1 + Fraction(1, 1 << 52)


# ---------------------------------------------------------------- BF16 rounding
def test_round_bf16_roundtrip_all_finite_patterns():
    allb = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    e = (allb >> 7) & 0xFF
    finite = allb[e != 0xFF]
    wide = oracle.widen_bf16(finite)
    # widening agrees with the field-by-field decode on a sample
    for b in finite[::997]:
        assert Fraction(float(oracle.widen_bf16(np.array([b], dtype=np.uint16))[0])) == frac_of_bits(int(b))
    assert np.array_equal(oracle.round_bf16(wide), finite)


def test_round_bf16_ties_to_even_and_neighbours():
    pos = np.arange(0x0000, 0x7F7F, dtype=np.uint16)  # finite positives incl. subnormals
    lo = oracle.widen_bf16(pos)
    hi = oracle.widen_bf16(pos + np.uint16(1))
    mid = (lo + hi) / 2.0
    even = np.where(pos & 1 == 0, pos, pos + np.uint16(1))
    assert np.array_equal(oracle.round_bf16(mid), even)
    assert np.array_equal(oracle.round_bf16(-mid), even | np.uint16(0x8000))
    just_below = np.nextafter(mid, 0.0)
    just_above = np.nextafter(mid, np.inf)
    assert np.array_equal(oracle.round_bf16(just_below), pos)
    assert np.array_equal(oracle.round_bf16(just_above), pos + np.uint16(1))


def test_round_bf16_specials_and_library_agreement():
    big = oracle.widen_bf16(np.array([0x7F7F], dtype=np.uint16))[0]
    ulp = 2.0 ** (127 - 7)
    assert oracle.round_bf16(np.array([big + ulp / 2]))[0] == 0x7F80      # tie -> even -> inf
    assert oracle.round_bf16(np.array([np.nextafter(big + ulp / 2, 0)]))[0] == 0x7F7F
    assert oracle.round_bf16(np.array([np.inf, -np.inf])).tolist() == [0x7F80, 0xFF80]
    assert oracle.round_bf16(np.array([0.0, -0.0])).tolist() == [0x0000, 0x8000]
    n = oracle.round_bf16(np.array([np.nan]))[0]
    assert (n & 0x7F80) == 0x7F80 and (n & 0x7F) != 0
    # float32-representable doubles: a single rounding either way, so the
    # library's float32 -> bfloat16 conversion must agree bit for bit
    g = np.random.Generator(np.random.Philox(key=[1, 2]))
    v = (g.standard_normal(200000, dtype=np.float32) * np.float32(3.0))
    v[:1000] *= np.float32(1e-39)   # subnormal range
    t = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.round_bf16(v.astype(np.float64)), t)


def test_bad_arguments_are_rejected():
    X = np.zeros((2, 4), dtype=np.uint16)
    W = np.zeros((3, 4), dtype=np.uint16)
    with pytest.raises(ValueError):
        oracle.outproj(X, W, np.zeros(4, dtype=np.uint16))
    with pytest.raises(TypeError):
        oracle.outproj(X.astype(np.float32), W)
    with pytest.raises(RuntimeError):
        oracle.outproj_rows(X, W, None, None, np.array([2]))
