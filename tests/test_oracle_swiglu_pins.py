"""Pins for the oracle's gate/up + SwiGLU: its two projections against the (separately
pinned) plain projection and a float64 library matmul, its activation against exact
identities and a float64 library silu, and closed forms that fix which operand is gated."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_17071_b200 import inputs
from test_oracle_pins import bits


def f64(b):
    return inputs.bf16_bits_to_f32(b).astype(np.float64)


def case(M, I, K, seed=3, std=1.0):
    X = inputs.normal_bf16(seed, "X", (M, K), std)
    Wg = inputs.normal_bf16(seed, "W", (I, K), 1.0 / np.sqrt(K))
    Wu = inputs.normal_bf16(seed + 1, "W", (I, K), 1.0 / np.sqrt(K))
    return X, Wg, Wu


def test_projections_are_the_plain_projections():
    X, Wg, Wu = case(9, 14, 40)
    z, g, u = oracle.swiglu(X, Wg, Wu, want_parts=True)
    assert np.array_equal(g, oracle.outproj(X, Wg)) and np.array_equal(u, oracle.outproj(X, Wu))
    Xd, Gd, Ud = (torch.from_numpy(f64(a)) for a in (X, Wg, Wu))
    lib = (torch.nn.functional.silu(Xd @ Gd.T) * (Xd @ Ud.T)).numpy()
    assert np.max(np.abs(z - lib)) <= 1e-13 * max(1.0, np.abs(lib).max())
    rows = np.array([8, 0, 3, 3])
    assert np.array_equal(oracle.swiglu(X, Wg, Wu, rows=rows), z[rows])


def test_activation_identities():
    """With K = 1, X = 1 the pre-activations are the weights themselves, so z = silu(wg) * wu
    elementwise: check silu(t) - silu(-t) = t (exact identity), silu(0) = 0, the large-|t|
    limits and monotone growth for t > 0."""
    t = np.array([0.0, 0.5, 1.0, 2.0, 3.5, 8.0, 30.0, 90.0, -0.5, -1.0, -2.0, -3.5, -8.0, -30.0, -90.0])
    X = bits(np.ones((1, 1)))
    Wg = bits(t.reshape(-1, 1))
    one = bits(np.ones((len(t), 1)))
    s = oracle.swiglu(X, Wg, one)[0]
    tt = f64(Wg)[:, 0]
    for a in (0.5, 1.0, 2.0, 3.5, 8.0, 30.0):
        sp, sn = s[list(tt).index(a)], s[list(tt).index(-a)]
        assert sp - sn == pytest.approx(a, rel=1e-15)
    assert s[0] == 0.0
    assert s[list(tt).index(90.0)] == pytest.approx(90.0, rel=1e-15)
    assert abs(s[list(tt).index(-90.0)]) < 1e-35
    pos = s[1:8]
    assert (np.diff(pos) > 0).all()
    # the second factor multiplies linearly and it is Wg, not Wu, that goes through silu
    Wu = bits(np.full((len(t), 1), -4.0))
    assert np.allclose(oracle.swiglu(X, Wg, Wu)[0], -4.0 * s, rtol=1e-15)
    swapped = oracle.swiglu(X, Wu, Wg)[0]
    assert not np.allclose(swapped, -4.0 * s)


def test_closed_forms_and_invariants():
    M, I, K = 6, 10, 24
    X, Wg, Wu = case(M, I, K, seed=9)
    z = oracle.swiglu(X, Wg, Wu)
    zero = np.zeros((I, K), dtype=np.uint16)
    assert not oracle.swiglu(X, zero, Wu).any()            # silu(0) = 0
    assert not oracle.swiglu(X, Wg, zero).any()
    Wu2 = bits(2.0 * inputs.bf16_bits_to_f32(Wu))
    assert np.array_equal(oracle.swiglu(X, Wg, Wu2), 2.0 * z)   # linear in the up projection
    # one-hot rows of X pick one column of each weight: z[m,i] = silu(Wg[i,m]) * Wu[i,m]
    X1 = inputs.one_hot_rows_bf16(M, K)
    g, u = f64(Wg)[:, :M].T, f64(Wu)[:, :M].T
    want = torch.nn.functional.silu(torch.from_numpy(g)).numpy() * u
    assert np.allclose(oracle.swiglu(X1, Wg, Wu), want, rtol=1e-14, atol=0)


def test_bad_arguments():
    X, Wg, Wu = case(2, 3, 8)
    with pytest.raises(ValueError):
        oracle.swiglu(X, Wg, Wu[:2])
    with pytest.raises(RuntimeError):
        oracle.swiglu(X, Wg, Wu, rows=np.array([5]))
