"""Parity at the full sizes of the measured workloads, in the launch
configuration the benchmark times (public entry points, automatic plan).  The
oracle computes a deterministic stratified sample of rows (every 128-row block
contributes two rows, all columns) exactly; small-M shapes are checked whole."""
import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu

NAMES = ["cfg1", "cfg2", "cfg4", "cfg5", "gemm4096"] + [w.name for w in inputs.sweep_workloads()]


@pytest.mark.parametrize("name", NAMES)
def test_full_size_workload(name):
    wl = inputs.all_workloads()[name]
    d = inputs.make_inputs(wl)
    X, W, b, R = d["X"], d["W"], d["bias"], d["R"]
    Xd, Wd, bd, Rd = kt.to_dev(X), kt.to_dev(W), kt.to_dev(b), kt.to_dev(R)
    Y = kt.nan_filled(wl.M, wl.N)
    if wl.has_residual:
        kx.kx_outproj_residual(Xd, Wd, bd, Rd, Y)
    else:
        kx.kx_gemm_bf16(Xd, Wd, Y)
    code, detail = kx.kx_last_device_status()
    assert code == kx.KX_OK, (code, detail)
    y = kt.from_dev(Y)
    assert not np.isnan(oracle.widen_bf16(y)).any(), "unwritten outputs"
    rows = None if wl.M <= 128 else inputs.sampled_rows(wl.M)
    ref, absref = oracle.outproj_rows(X, W, b, R, rows, want_abs=True)
    ys = y if rows is None else y[rows]
    ok, msg = kt.gate_a(ys, ref)
    assert ok, f"{name}: {msg}"
    ok, msg = kt.gate_c(ys, ref, absref, wl.K, rate_limit=5e-3 if wl.has_residual else 3e-2)
    assert ok, f"{name}: {msg}"
    if not wl.has_residual:
        assert kt.rel_fro(ys, ref) <= 2.0 ** -8
    # in place (output aliased onto the residual) gives the same bits
    if wl.has_residual:
        kx.kx_outproj_residual(Xd, Wd, bd, Rd, Rd)
        assert np.array_equal(kt.from_dev(Rd), y)
    # a few single elements computed one by one
    g = np.random.Generator(np.random.Philox(key=[wl.seed, 99]))
    for _ in range(4):
        m, n = int(g.integers(0, wl.M)), int(g.integers(0, wl.N))
        r = oracle.element(X, W, b, R, m, n)
        yv = oracle.widen_bf16(y[m:m + 1, n:n + 1])[0, 0]
        assert abs(yv - r) <= kt.ATOL + kt.RTOL * abs(r), (name, m, n, yv, r)


def test_exact_integer_arithmetic_at_full_size():
    """Ternary operands at the largest shapes: bit-exact on sampled rows."""
    for (M, N, K) in [(4096, 4096, 4096), (16384, 4096, 14336), (512, 8192, 8192), (32, 8192, 8192)]:
        X = inputs.ternary_bf16(3, "X", (M, K))
        W = inputs.ternary_bf16(3, "W", (N, K))
        b = inputs.small_int_bf16(3, "bias", (N,), -4, 4)
        R = inputs.small_int_bf16(3, "R", (M, N), -8, 8)
        Y = kt.nan_filled(M, N)
        kx.kx_outproj_residual(kt.to_dev(X), kt.to_dev(W), kt.to_dev(b), kt.to_dev(R), Y)
        assert kx.kx_last_device_status()[0] == kx.KX_OK
        y = kt.from_dev(Y)
        rows = None if M <= 128 else inputs.sampled_rows(M)
        ref, _ = oracle.outproj_rows(X, W, b, R, rows)
        ok, msg = kt.gate_exact(y if rows is None else y[rows], ref)
        assert ok, f"{(M, N, K)}: {msg}"
