"""Seeded random shapes through every kernel variant: ternary operands (every partial sum an exact
integer), so any plan must reproduce the once-rounded exact result bit for bit.  Shapes are drawn
to hit ragged row / column / reduction tails, one-stage and odd-stage segments, single- and
multi-wave grids (through `max_ctas`), K clusters, half-width tails and stream-K."""
import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt
from test_gpu_parity import run, ternary_case, TILE_VARIANTS, SWAP_VARIANTS, STREAMK_VARIANTS, T

pytestmark = pytest.mark.gpu


def draw_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    extra = [dict(path=T, block_n=256, cta_pair=1, k_cluster=2), dict(path=T, block_n=128, cta_pair=1, k_cluster=2, stages=3),
             dict(path=T, block_n=192, cta_pair=1, k_cluster=4), dict(path=T, block_n=256, cta_pair=2, narrow_tail=2, stages=3),
             dict(path=T, block_n=128, cta_pair=1, narrow_tail=2), dict(path=T, block_n=256, cta_pair=2, k_cluster=2),
             dict(path=T, block_n=128, cta_pair=2, k_cluster=2, stages=4), dict(path=T, block_n=256, cta_pair=2, stream_k=3),
             dict(path=T, block_n=128, cta_pair=1, stream_k=3, stages=3), None]
    pool = TILE_VARIANTS + SWAP_VARIANTS + STREAMK_VARIANTS + extra
    while len(cases) < n:
        ov = pool[int(rng.integers(0, len(pool)))]
        small = ov is not None and ov.get("path") != T
        M = int(rng.integers(1, 65 if small else 900))
        N = 8 * int(rng.integers(1, 140))
        K = 8 * int(rng.integers(1, 180))
        o = dict(ov) if ov else {}
        if not small and rng.random() < 0.5:
            o["max_ctas"] = int(rng.choice([2, 4, 6, 10, 37]))
        if small and M > o.get("block_n", 256) * 4:
            continue
        try:
            kx.kx_plan_query(M, N, K, ov=kx.make_override(**o) if o else None)
        except kx.KxError:
            continue                                   # not a valid plan for this shape (e.g. K cluster on a short K)
        cases.append((M, N, K, o))
    return cases


@pytest.mark.parametrize("chunk", range(12))
def test_random_shapes_and_plans_are_exact(chunk):
    for (M, N, K, o) in draw_cases(20, 1000 + chunk):
        X, W, b, R = ternary_case(M, N, K, seed=chunk)
        y = run(X, W, b, R, o or None)
        ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
        assert ok, f"M={M} N={N} K={K} plan={o}: {msg}"
