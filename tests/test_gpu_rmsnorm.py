"""RMSNorm after the output projection: the CUDA kernel against the CPU oracle, alone
(on exactly the same BF16 input bits) and chained after the projection."""
import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu


def gate_norm(z_bits, ref):
    """One BF16 rounding (half an ulp = 2^-9 relative) plus FP32 arithmetic (sum of squares,
    rsqrt, two products: < 2^-18 relative): allow one full ulp, 2^-8 relative."""
    z = oracle.widen_bf16(z_bits)
    assert not np.isnan(z).any()
    err = np.abs(z - ref)
    allow = 2.0 ** -8 * np.abs(ref) + 1e-37
    assert (err <= allow).all(), float((err / allow).max())
    rate = float((oracle.round_bf16(ref) != z_bits).mean())
    assert rate <= 0.01, rate


@pytest.mark.parametrize("M,N", [(1, 8), (3, 264), (130, 4096), (17, 32768), (1000, 5120), (2500, 2048), (7, 3072), (3, 8192), (5, 6144), (9, 7168), (5, 2560), (9000, 256)])
@pytest.mark.parametrize("eps", [1e-6, 0.0])
def test_rmsnorm_matches_oracle(M, N, eps):
    H = inputs.normal_bf16(200 + N, "R", (M, N), 1.0)
    g = inputs.normal_bf16(200 + N, "bias", (N,), 1.0)
    Z = kt.nan_filled(M, N)
    kx.kx_rmsnorm(kt.to_dev(H), kt.to_dev(g), eps, Z)
    z = kt.from_dev(Z)
    gate_norm(z, oracle.rmsnorm(H, g, eps))
    # in place gives the same bits
    Hd = kt.to_dev(H)
    kx.kx_rmsnorm(Hd, kt.to_dev(g), eps, Hd)
    assert np.array_equal(kt.from_dev(Hd), z)


def test_rmsnorm_exact_cases():
    N = 1024
    one = inputs.f32_to_bf16_bits(np.ones(N, dtype=np.float32))
    # constant power-of-two rows, gamma = 1, eps = 0: z = sign(c) exactly after rounding
    H = inputs.f32_to_bf16_bits(np.repeat(np.array([[0.25], [-8.0], [1.0]], dtype=np.float32), N, axis=1))
    Z = kt.nan_filled(3, N)
    kx.kx_rmsnorm(kt.to_dev(H), kt.to_dev(one), 0.0, Z)
    z = oracle.widen_bf16(kt.from_dev(Z))
    assert (z[0] == 1.0).all() and (z[1] == -1.0).all() and (z[2] == 1.0).all()
    # a zero row with eps > 0 stays zero; rows are independent
    H2 = inputs.normal_bf16(5, "R", (4, N), 1.0)
    H2[2] = 0
    Z = kt.nan_filled(4, N)
    kx.kx_rmsnorm(kt.to_dev(H2), kt.to_dev(one), 1e-6, Z)
    z2 = kt.from_dev(Z)
    assert not (z2[2] & 0x7FFF).any()
    Z1 = kt.nan_filled(1, N)
    kx.kx_rmsnorm(kt.to_dev(H2[3:4].copy()), kt.to_dev(one), 1e-6, Z1)
    assert np.array_equal(kt.from_dev(Z1)[0], z2[3])


@pytest.mark.parametrize("M,N,K", [(32, 2048, 2048), (700, 1032, 520), (128, 1024, 1024)])
def test_projection_then_rmsnorm(M, N, K):
    d = inputs.make_inputs(inputs.Workload("t", M, N, K, 301, True, True), stress=True)
    g = inputs.normal_bf16(301, "X", (N,), 1.0)
    X, W, b, R = (kt.to_dev(d[k]) for k in ("X", "W", "bias", "R"))
    H, Z = kt.nan_filled(M, N), kt.nan_filled(M, N)
    kx.kx_outproj_residual_rmsnorm(X, W, b, R, kt.to_dev(g), 1e-5, H, Z)
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    h, z = kt.from_dev(H), kt.from_dev(Z)
    # H is exactly what the projection alone writes
    Y = kt.nan_filled(M, N)
    kx.kx_outproj_residual(X, W, b, R, Y)
    assert np.array_equal(kt.from_dev(Y), h)
    ref_h = oracle.outproj(d["X"], d["W"], d["bias"], d["R"])
    ok, msg = kt.gate_a(h, ref_h)
    assert ok, msg
    # Z against the oracle's RMSNorm of the very bits the kernel normalised (sharp) ...
    gate_norm(z, oracle.rmsnorm(h, g, 1e-5))
    # ... and against the all-oracle chain (H rounded once from the FP64 sum): the two H can
    # differ in the last BF16 bit where FP32 accumulation straddles a rounding boundary
    ref_z = oracle.rmsnorm(oracle.round_bf16(ref_h), g, 1e-5)
    ok, msg = kt.gate_a(z, ref_z)
    assert ok, msg
    # in-place residual stream (H aliased onto R) gives the same H and Z
    Rd = kt.to_dev(d["R"])
    Z2 = kt.nan_filled(M, N)
    kx.kx_outproj_residual_rmsnorm(X, W, b, Rd, kt.to_dev(g), 1e-5, Rd, Z2)
    assert np.array_equal(kt.from_dev(Rd), h) and np.array_equal(kt.from_dev(Z2), z)


def test_projection_then_rmsnorm_full_size():
    wl = inputs.all_workloads()["cfg2"]
    d = inputs.make_inputs(wl)
    g = inputs.normal_bf16(wl.seed, "bias", (wl.N,), 1.0)
    H, Z = kt.nan_filled(wl.M, wl.N), kt.nan_filled(wl.M, wl.N)
    kx.kx_outproj_residual_rmsnorm(kt.to_dev(d["X"]), kt.to_dev(d["W"]), None, kt.to_dev(d["R"]), kt.to_dev(g),
                                   1e-6, H, Z)
    assert kx.kx_last_device_status()[0] == kx.KX_OK
    h, z = kt.from_dev(H), kt.from_dev(Z)
    rows = inputs.sampled_rows(wl.M)
    ref_h, _ = oracle.outproj_rows(d["X"], d["W"], None, d["R"], rows)
    ok, msg = kt.gate_a(h[rows], ref_h)
    assert ok, msg
    gate_norm(z[rows], oracle.rmsnorm(h, g, 1e-6, rows=rows))
