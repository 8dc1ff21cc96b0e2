"""Bounded device-side waits: a wait that can never complete gives up after its
limit, the kernel exits cleanly (TMEM freed, context usable) and the host reads
KX_ERR_DEVICE_TIMEOUT.  The wait is made to run out from the host side: the plan
override tells the TMA producer to issue one k-block fewer than the MMA consumer
expects, so the consumer waits on a barrier that nothing completes.  No trap, no
bad address, no unbounded loop is involved."""
import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu

T, S = kx.KX_PATH_TILE, kx.KX_PATH_SWAP
WAIT_FULL = 2   # the MMA issuer's wait for a filled stage


@pytest.mark.parametrize("ov", [dict(path=T, block_n=256, cta_pair=1), dict(path=T, block_n=128, cta_pair=2),
                                dict(path=S, block_n=128, split_k=2),
                                dict(path=T, block_n=256, cta_pair=2, stream_k=2),
                                dict(path=T, block_n=128, cta_pair=1, k_cluster=2),
                                dict(path=S, block_n=128, split_k=2, cluster_reduce=1),
                                dict(path=S, block_n=128, split_k=2, cluster_reduce=2),
                                dict(path=S, block_n=32, split_k=4, cluster_reduce=3),
                                dict(path=T, block_n=256, cta_pair=2, k_cluster=2),
                                dict(path=T, block_n=128, cta_pair=1, stream_k=3, max_ctas=3),
                                dict(path=T, block_n=128, cta_pair=1, narrow_tail=3, max_ctas=3)],
                         ids=["tile", "pair", "swap-cluster", "pair-streamk", "tile-kcluster", "swap-workspace",
                              "swap-cluster-pull", "swap-cluster-push", "pair-kcluster", "streamk-first", "k-halves"])
def test_wait_gives_up_and_context_survives(ov):
    import time
    M, N, K = (128 if ov.get("block_n", 0) >= 128 else 30), 512, 512
    X = inputs.ternary_bf16(1, "X", (M, K))
    W = inputs.ternary_bf16(1, "W", (N, K))
    R = inputs.small_int_bf16(1, "R", (M, N), -8, 8)
    Xd, Wd, Rd = kt.to_dev(X), kt.to_dev(W), kt.to_dev(R)
    Y = kt.nan_filled(M, N)
    bad = kx.make_override(debug_drop_kblocks=1, spin_limit_us=20000, **ov)
    t0 = time.time()
    assert kx.kx_outproj_residual_ex(Xd, Wd, None, Rd, Y, bad) == kx.KX_OK   # the launch itself succeeds
    code, detail = kx.kx_last_device_status()
    assert code == kx.KX_ERR_DEVICE_TIMEOUT and detail == WAIT_FULL
    assert time.time() - t0 < 5.0
    assert kx.kx_last_device_status() == (kx.KX_OK, 0)                      # reading clears it
    # the same context runs the same plan correctly afterwards (counters were reset)
    for _ in range(2):
        Y = kt.nan_filled(M, N)
        kx.kx_outproj_residual_ex(Xd, Wd, None, Rd, Y, kx.make_override(**ov))
        assert kx.kx_last_device_status() == (kx.KX_OK, 0)
        ok, msg = kt.gate_exact(kt.from_dev(Y), oracle.outproj(X, W, None, R))
        assert ok, msg
