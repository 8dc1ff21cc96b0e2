"""The seeded input generator: reproducible, independent streams, the stated
distributions, and a BF16 packing that agrees with a library conversion."""
import math

import numpy as np
import torch

from paper_2608_17071_b200 import inputs


def test_bf16_packing_matches_library():
    g = np.random.Generator(np.random.Philox(key=[9, 9]))
    v = g.standard_normal(100000, dtype=np.float32)
    t = torch.from_numpy(v).to(torch.bfloat16)
    assert np.array_equal(inputs.f32_to_bf16_bits(v), t.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(v)), t.float().numpy())
    assert inputs.f32_to_bf16_bits(np.array([np.nan], dtype=np.float32))[0] == 0x7FC0


def test_reproducible_and_independent():
    a = inputs.normal_bf16(3, "X", (64, 32), 1.0)
    b = inputs.normal_bf16(3, "X", (64, 32), 1.0)
    c = inputs.normal_bf16(3, "W", (64, 32), 1.0)
    d = inputs.normal_bf16(4, "X", (64, 32), 1.0)
    assert np.array_equal(a, b)
    assert not np.array_equal(a, c) and not np.array_equal(a, d)
    # a prefix of a longer draw of the same stream is the same data
    e = inputs.normal_bf16(3, "X", (128, 32), 1.0)
    assert np.array_equal(e[:64], a)


def test_distributions():
    wl = inputs.all_workloads()["cfg1"]
    d = inputs.make_inputs(wl)
    f = inputs.bf16_bits_to_f32
    assert d["X"].shape == (128, 1024) and d["W"].shape == (1024, 1024)
    assert d["bias"].shape == (1024,) and d["R"].shape == (128, 1024)
    assert abs(f(d["X"]).std() * math.sqrt(1024) - 1) < 0.02
    assert abs(f(d["W"]).std() * math.sqrt(1024) - 1) < 0.02
    assert abs(f(d["R"]).std() - 1) < 0.02 and abs(f(d["R"]).mean()) < 0.02
    assert abs(f(d["bias"]).std() - 0.1) < 0.01
    s = inputs.make_inputs(wl, stress=True)
    assert abs(f(s["X"]).std() - 1) < 0.02
    u = inputs.uniform_bf16(20, "X", (256, 256), 1.0 / 16)
    uf = f(u)
    assert uf.min() >= -1 / 16 and uf.max() <= 1 / 16 and abs(uf.std() * 16 - 1 / math.sqrt(3)) < 0.01


def test_workload_table():
    w = inputs.all_workloads()
    assert (w["cfg2"].M, w["cfg2"].N, w["cfg2"].K, w["cfg2"].seed) == (4096, 4096, 4096, 1)
    assert not w["cfg2"].has_bias and w["cfg2"].has_residual
    assert (w["cfg5"].M, w["cfg5"].N, w["cfg5"].K) == (16384, 4096, 14336)
    assert w["cfg4"].dist == "uniform" and not w["cfg4"].has_residual
    sw = inputs.sweep_workloads()
    assert len(sw) == 16 and [s.seed for s in sw] == list(range(2, 18))
    assert (sw[0].M, sw[0].K) == (1, 2048) and (sw[5].M, sw[5].K) == (32, 4096) and (sw[15].M, sw[15].N) == (8192, 8192)
    assert w["cfg2"].flops == 2 * 4096 ** 3
    assert w["cfg2"].algorithmic_bytes == 2 * 4 * 4096 ** 2


def test_structured_inputs():
    t = inputs.bf16_bits_to_f32(inputs.ternary_bf16(1, "X", (50, 50)))
    assert set(np.unique(t).tolist()) == {-1.0, 0.0, 1.0}
    W, pi = inputs.permutation_matrix_bf16(2, 10, 16)
    Wf = inputs.bf16_bits_to_f32(W)
    assert (Wf.sum(axis=1) == 1).all() and len(set(pi.tolist())) == 10
    assert all(Wf[n, pi[n]] == 1 for n in range(10))
    X = inputs.bf16_bits_to_f32(inputs.one_hot_rows_bf16(5, 3))
    assert X[4, 1] == 1 and X.sum() == 5
