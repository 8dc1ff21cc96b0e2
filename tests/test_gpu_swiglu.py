"""Gate/up projections with the fused SwiGLU epilogue against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu


def make(M, I, K, seed, xstd=1.0):
    X = inputs.normal_bf16(seed, "X", (M, K), xstd)
    Wg = inputs.normal_bf16(seed, "W", (I, K), 1.0 / np.sqrt(K))
    Wu = inputs.normal_bf16(seed + 1, "W", (I, K), 1.0 / np.sqrt(K))
    return X, Wg, Wu


def run(X, Wg, Wu):
    M, I = X.shape[0], Wg.shape[0]
    Z = kt.nan_filled(M, I)
    kx.kx_gate_up_swiglu(kt.to_dev(X), kt.to_dev(Wg), kt.to_dev(Wu), Z)
    code, detail = kx.kx_last_device_status()
    assert code == kx.KX_OK, (code, detail)
    return kt.from_dev(Z)


def check(z_bits, ref):
    ok, msg = kt.gate_a(z_bits, ref)
    assert ok, msg
    assert kt.rel_fro(z_bits, ref) <= 2.0 ** -8
    # one BF16 rounding plus FP32 accumulation / activation error: within one ulp-ish
    z = oracle.widen_bf16(z_bits)
    assert (np.abs(z - ref) <= 2.0 ** -7 * np.abs(ref) + 2e-3).all()


# single-CTA tiles (few tiles) and CTA-pair tiles (enough 256-row tiles to fill the pair slots)
@pytest.mark.parametrize("M,I,K", [(128, 128, 64), (300, 520, 264), (640, 1024, 512), (7, 776, 1096),
                                   (2048, 4096, 512), (2500, 3080, 264)])
def test_swiglu_matches_oracle(M, I, K):
    X, Wg, Wu = make(M, I, K, seed=400 + M)
    check(run(X, Wg, Wu), oracle.swiglu(X, Wg, Wu))


def test_swiglu_long_reduction():
    X, Wg, Wu = make(256, 256, 14336, seed=410)
    check(run(X, Wg, Wu), oracle.swiglu(X, Wg, Wu))


@pytest.mark.parametrize("M,I,K", [(384, 520, 320), (2048, 4096, 256)])
def test_swiglu_exact_pins(M, I, K):
    """Properties that hold bit for bit whatever the summation order."""
    X, Wg, Wu = make(M, I, K, seed=420)
    z = run(X, Wg, Wu)
    zero = np.zeros_like(Wg)
    assert not (run(X, zero, Wu) & 0x7FFF).any()           # silu(0) * u = 0
    assert not (run(X, Wg, zero) & 0x7FFF).any()           # silu(g) * 0 = 0
    Wu2 = inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(Wu))
    want = inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(z))
    assert np.array_equal(run(X, Wg, Wu2), want)            # linear in the up projection
    assert np.array_equal(run(X, Wg, Wu), z)                # deterministic


def test_swiglu_selectors_fix_the_gate_up_pairing():
    """One-hot rows of X: z[m,i] = silu(Wg[i, m mod K]) * Wu[i, m mod K]; a swapped or shifted
    gate/up pairing in the epilogue would be off by O(1)."""
    M, I, K = 260, 392, 448
    X = inputs.one_hot_rows_bf16(M, K)
    Wg = inputs.normal_bf16(430, "W", (I, K), 1.0)
    Wu = inputs.normal_bf16(431, "W", (I, K), 1.0)
    z = oracle.widen_bf16(run(X, Wg, Wu))
    ref = oracle.swiglu(X, Wg, Wu)
    assert (np.abs(z - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-6).all()
    g = oracle.widen_bf16(Wg)[:, np.arange(M) % K].T
    u = oracle.widen_bf16(Wu)[:, np.arange(M) % K].T
    assert np.allclose(ref, g / (1.0 + np.exp(-g)) * u, rtol=1e-12)


def test_swiglu_edge_cases_and_errors():
    X, Wg, Wu = make(5, 16, 8, seed=440)
    check(run(X, Wg, Wu), oracle.swiglu(X, Wg, Wu))
    Z = kt.nan_filled(5, 16)
    assert kx.kx_gate_up_swiglu(0, 0, 0, Z, M=5, I=16, K=0) == kx.KX_OK      # empty sums
    assert not kt.from_dev(Z).any()
    A = 0x10000
    assert kx.kx_gate_up_swiglu(A, A * 4, A * 8, A * 16, M=4, I=12, K=8, check=False) == kx.KX_ERR_SHAPE
    assert kx.kx_gate_up_swiglu(A, A * 4, A * 8, A, M=4, I=8, K=8, check=False) == kx.KX_ERR_OVERLAP
    assert kx.kx_gate_up_swiglu(A, 0, A * 8, A * 16, M=4, I=8, K=8, check=False) == kx.KX_ERR_NULL


def test_swiglu_full_size_sampled_rows():
    """The gate/up GEMM that feeds the 14336 -> 4096 down projection: M = 4096 tokens."""
    M, I, K = 4096, 14336, 4096
    X, Wg, Wu = make(M, I, K, seed=450, xstd=1.0)
    z = run(X, Wg, Wu)
    assert not np.isnan(oracle.widen_bf16(z)).any()
    rows = inputs.sampled_rows(M)[::4]
    check(z[rows], oracle.swiglu(X, Wg, Wu, rows=rows))
