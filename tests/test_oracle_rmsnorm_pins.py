"""Pins for the oracle's RMSNorm: exact rational brute force, closed forms, invariances
and a float64 library routine — none of them the oracle's own formula retyped."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import inputs
from test_oracle_pins import bits, frac_of_bits


@pytest.mark.parametrize("M,N", [(1, 1), (3, 8), (5, 17), (2, 64)])
@pytest.mark.parametrize("eps", [0.0, 1e-6, 0.5])
def test_squared_identity_in_exact_arithmetic(M, N, eps):
    """z^2 * (mean(h^2) + eps) == h^2 * gamma^2 with the mean of squares taken exactly
    (rational arithmetic on the decoded BF16 values); also pins the sign of z."""
    H = inputs.normal_bf16(50 + N, "X", (M, N), 1.0)
    g = inputs.normal_bf16(51 + N, "bias", (N,), 1.0)
    z = oracle.rmsnorm(H, g, eps)
    for m in range(M):
        hs = [frac_of_bits(int(H[m, j])) for j in range(N)]
        ms = sum(h * h for h in hs) / N + Fraction(eps)
        for j in range(N):
            gj = frac_of_bits(int(g[j]))
            want2 = hs[j] * hs[j] * gj * gj
            got2 = Fraction(float(z[m, j])) ** 2 * ms
            assert abs(got2 - want2) <= want2 * Fraction(1, 1 << 48) + Fraction(1, 10 ** 300)
            assert (z[m, j] > 0) == (hs[j] * gj > 0) and (z[m, j] < 0) == (hs[j] * gj < 0)


def test_closed_forms():
    N = 40
    g = bits(np.linspace(-2, 2, N))
    gf = inputs.bf16_bits_to_f32(g).astype(np.float64)
    # constant row c, eps = 0: z = sign(c) * gamma
    for c in (0.5, -3.0, 128.0):
        z = oracle.rmsnorm(bits(np.full((1, N), c)), g, 0.0)
        assert np.allclose(z[0], np.sign(c) * gf, rtol=1e-15, atol=0)
    # one non-zero element a at column 7: mean of squares = a^2 / N, so z_7 = sqrt(N) * sign(a) * gamma_7
    h = np.zeros((1, N)); h[0, 7] = -4.0
    z = oracle.rmsnorm(bits(h), g, 0.0)
    assert z[0, 7] == pytest.approx(-np.sqrt(N) * gf[7], rel=1e-15) and np.count_nonzero(z) == 1
    # eps dominates: h = 2^-60 tiny, eps = 1 -> z = h * gamma (to 1e-30)
    h = np.full((1, N), 2.0 ** -60)
    z = oracle.rmsnorm(bits(h), g, 1.0)
    assert np.allclose(z[0], 2.0 ** -60 * gf, rtol=1e-15)
    # all-zero row with eps > 0 gives zeros, not NaN
    assert not oracle.rmsnorm(bits(np.zeros((2, N))), g, 1e-6).any()


def test_invariances():
    M, N = 6, 96
    H = inputs.normal_bf16(60, "X", (M, N), 1.0)
    g = inputs.normal_bf16(60, "bias", (N,), 1.0)
    z = oracle.rmsnorm(H, g, 0.0)
    # scaling a row by a power of two does not change z when eps = 0
    H4 = bits(4.0 * inputs.bf16_bits_to_f32(H))
    assert np.allclose(oracle.rmsnorm(H4, g, 0.0), z, rtol=1e-15)
    # rows are independent and `rows` selects them
    rr = np.array([5, 0, 0, 3])
    assert np.array_equal(oracle.rmsnorm(H, g, 0.0, rows=rr), z[rr])
    # permuting columns of h and gamma together permutes z
    perm = np.random.Generator(np.random.Philox(key=[7, 7])).permutation(N)
    zp = oracle.rmsnorm(np.ascontiguousarray(H[:, perm]), np.ascontiguousarray(g[perm]), 0.0)
    assert np.allclose(zp, z[:, perm], rtol=1e-14)
    # with gamma = 1 and eps = 0 every row of z has mean square exactly 1
    one = bits(np.ones(N))
    z1 = oracle.rmsnorm(H, one, 0.0)
    assert np.allclose((z1 ** 2).mean(axis=1), 1.0, rtol=1e-14)
    # gamma enters linearly
    g2 = bits(2.0 * inputs.bf16_bits_to_f32(g))
    assert np.allclose(oracle.rmsnorm(H, g2, 1e-5), 2.0 * oracle.rmsnorm(H, g, 1e-5), rtol=1e-15)


@pytest.mark.parametrize("eps", [1e-6, 1e-5])
def test_against_float64_library_rms_norm(eps):
    M, N = 33, 1032
    H = inputs.normal_bf16(70, "X", (M, N), 1.0)
    g = inputs.normal_bf16(70, "bias", (N,), 0.5)
    Hd = torch.from_numpy(inputs.bf16_bits_to_f32(H).astype(np.float64))
    gd = torch.from_numpy(inputs.bf16_bits_to_f32(g).astype(np.float64))
    lib = torch.nn.functional.rms_norm(Hd, (N,), weight=gd, eps=eps).numpy()
    z = oracle.rmsnorm(H, g, eps)
    assert np.max(np.abs(z - lib)) <= 1e-13 * max(1.0, np.max(np.abs(lib)))


def test_bad_arguments():
    H = np.zeros((2, 8), dtype=np.uint16)
    with pytest.raises(ValueError):
        oracle.rmsnorm(H, np.zeros(4, dtype=np.uint16), 0.0)
    with pytest.raises(RuntimeError):
        oracle.rmsnorm(H, np.zeros(8, dtype=np.uint16), 0.0, rows=np.array([2]))
