"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by
element, on sizes the oracle finishes in seconds: every kernel variant, several
tiles plus ragged tails, exact pins and the tolerance gates."""
import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu

T, S = kx.KX_PATH_TILE, kx.KX_PATH_SWAP
TILE_VARIANTS = [
    dict(path=T, block_n=256, cta_pair=1), dict(path=T, block_n=128, cta_pair=1),
    dict(path=T, block_n=64, cta_pair=1), dict(path=T, block_n=256, cta_pair=2),
    dict(path=T, block_n=128, cta_pair=2), dict(path=T, block_n=192, cta_pair=1),
    dict(path=T, block_n=192, cta_pair=2),
    # the variants with two k-blocks per ring stage (selected by their stage count)
    dict(path=T, block_n=256, cta_pair=2, stages=3), dict(path=T, block_n=256, cta_pair=1, stages=2),
    dict(path=T, block_n=192, cta_pair=1, stages=2), dict(path=T, block_n=128, cta_pair=1, stages=3),
    dict(path=T, block_n=64, cta_pair=1, stages=4), dict(path=T, block_n=192, cta_pair=2, stages=3),
    dict(path=T, block_n=128, cta_pair=2, stages=4),
]
SWAP_VARIANTS = [
    dict(path=S, block_n=16, split_k=1), dict(path=S, block_n=16, split_k=4),
    dict(path=S, block_n=32, split_k=3), dict(path=S, block_n=64, split_k=2),
    dict(path=S, block_n=128, split_k=5), dict(path=S, block_n=256, split_k=1),
    dict(path=S, block_n=256, split_k=4),
    # the same split counts summed through the FP32 workspace instead of the cluster
    dict(path=S, block_n=16, split_k=4, cluster_reduce=1), dict(path=S, block_n=64, split_k=2, cluster_reduce=1),
    dict(path=S, block_n=256, split_k=4, cluster_reduce=1), dict(path=S, block_n=32, split_k=12),
    dict(path=S, block_n=128, split_k=8, cluster_reduce=2),
    # the variants with one k-block per ring stage (the defaults hold two)
    dict(path=S, block_n=16, split_k=4, stages=12), dict(path=S, block_n=32, split_k=3, stages=11, cluster_reduce=1),
    dict(path=S, block_n=64, split_k=2, stages=9), dict(path=S, block_n=128, split_k=5, stages=7), dict(path=S, block_n=256, split_k=1, stages=4),
    # cluster reduction with the partial rows pushed to their finishers (3) or pulled by them (2)
    dict(path=S, block_n=16, split_k=4, cluster_reduce=3), dict(path=S, block_n=32, split_k=3, cluster_reduce=3),
    dict(path=S, block_n=32, split_k=8, cluster_reduce=3), dict(path=S, block_n=64, split_k=2, cluster_reduce=3),
    dict(path=S, block_n=128, split_k=7, cluster_reduce=3), dict(path=S, block_n=32, split_k=3, cluster_reduce=2),
    dict(path=S, block_n=64, split_k=6, cluster_reduce=2),
]


def vid(v):
    return "-".join(f"{k}{val}" for k, val in v.items())


def run(X, W, b, R, ov=None, inplace=False, entry="ex"):
    M, K = X.shape
    N = W.shape[0]
    Xd, Wd, bd = kt.to_dev(X), kt.to_dev(W), kt.to_dev(b)
    if inplace:
        Y = kt.to_dev(R)
        Rd = Y
    else:
        Y = kt.nan_filled(M, N)
        Rd = kt.to_dev(R)
    o = kx.make_override(**ov) if ov else None
    if entry == "ex":
        kx.kx_outproj_residual_ex(Xd, Wd, bd, Rd, Y, o)
    elif entry == "fused":
        kx.kx_outproj_residual(Xd, Wd, bd, Rd, Y)
    else:
        kx.kx_gemm_bf16(Xd, Wd, Y)
    code, detail = kx.kx_last_device_status()
    assert code == kx.KX_OK, f"device status {code} (wait {detail})"
    return kt.from_dev(Y)


def ternary_case(M, N, K, seed=1, bias=True, res=True):
    X = inputs.ternary_bf16(seed, "X", (M, K))
    W = inputs.ternary_bf16(seed, "W", (N, K))
    b = inputs.small_int_bf16(seed, "bias", (N,), -4, 4) if bias else None
    R = inputs.small_int_bf16(seed, "R", (M, N), -8, 8) if res else None
    return X, W, b, R


# ------------------------------------------------------------------ exact pins
@pytest.mark.parametrize("ov", TILE_VARIANTS, ids=vid)
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (640, 1024, 512), (300, 520, 264), (1000, 776, 1096)])
def test_tile_exact_integer_arithmetic(ov, M, N, K):
    """X, W in {-1,0,1}, small-integer bias and residual: every partial sum is an
    integer below 2^24, FP32 accumulation is exact in any order, so the output
    must equal the once-rounded exact result bit for bit."""
    X, W, b, R = ternary_case(M, N, K)
    y = run(X, W, b, R, ov)
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg


@pytest.mark.parametrize("ov", SWAP_VARIANTS, ids=vid)
@pytest.mark.parametrize("N,K", [(256, 512), (1000, 1096), (2048, 4096)])
def test_swap_exact_integer_arithmetic(ov, N, K):
    bn = ov["block_n"]
    for M in sorted({1, bn // 2 + 1, bn, (2 * bn + 3) if bn >= 128 else bn}):
        X, W, b, R = ternary_case(M, N, K, seed=2)
        y = run(X, W, b, R, ov)
        ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
        assert ok, f"M={M}: {msg}"


STREAMK_VARIANTS = [
    dict(path=T, block_n=256, cta_pair=1, stream_k=2), dict(path=T, block_n=256, cta_pair=2, stream_k=2),
    dict(path=T, block_n=128, cta_pair=1, stream_k=2), dict(path=T, block_n=192, cta_pair=2, stream_k=2),
    dict(path=T, block_n=64, cta_pair=1, stream_k=2),
    # two k-blocks per ring stage: segments start at any k-block, stages pair up from there
    dict(path=T, block_n=256, cta_pair=2, stream_k=2, stages=3), dict(path=T, block_n=128, cta_pair=1, stream_k=2, stages=3),
]


@pytest.mark.parametrize("ov", STREAMK_VARIANTS, ids=vid)
@pytest.mark.parametrize("max_ctas", [0, 6, 37])
@pytest.mark.parametrize("M,N,K", [(640, 1024, 512), (300, 520, 264), (512, 2048, 2048), (1000, 776, 4096)])
def test_stream_k_exact_integer_arithmetic(ov, max_ctas, M, N, K):
    """Stream-K scheduling: every CTA takes an equal contiguous range of (tile, k-block)
    units, so tiles are split between CTAs at arbitrary k positions and summed through
    the workspace.  With integer-valued data the result must still be bit-exact, and
    the same bits must come out in place and on a second run (fixed summation order)."""
    X, W, b, R = ternary_case(M, N, K, seed=21)
    o = dict(ov, max_ctas=max_ctas)
    ref = oracle.outproj(X, W, b, R)
    y = run(X, W, b, R, o)
    ok, msg = kt.gate_exact(y, ref)
    assert ok, msg
    y2 = run(X, W, b, R.copy(), o, inplace=True)
    assert np.array_equal(y, y2)


@pytest.mark.parametrize("ov,max_ctas,M,N,K", [
    (dict(path=T, block_n=256, cta_pair=2), 12, 640, 1280, 520),     # 15 pair tiles on 6 slots: 3 split first, 12 whole
    (dict(path=T, block_n=256, cta_pair=2, stages=3), 12, 640, 1280, 4096),
    (dict(path=T, block_n=256, cta_pair=1), 10, 640, 1280, 1096),    # 25 tiles on 10 slots: 5 split first
    (dict(path=T, block_n=128, cta_pair=2), 12, 700, 520, 264),      # ragged rows and columns
    (dict(path=T, block_n=192, cta_pair=1, stages=2), 9, 300, 776, 2048),
    (dict(path=T, block_n=64, cta_pair=1), 37, 1000, 776, 520),
    (dict(path=T, block_n=256, cta_pair=2), 0, 4096, 2304, 264),     # full grid: 144 pair tiles on 74 slots
], ids=["pair256", "pair256-2kb-longk", "single256", "pair128-ragged", "single192-2kb", "single64", "pair256-fullgrid"])
def test_stream_k_first_exact_integer_arithmetic(ov, max_ctas, M, N, K):
    """The tiles left over after the full waves are cut into equal (tile, k-block) ranges and run first; the slot
    that ends a split tile last adds the parked partials in fixed order while the next whole tile is in its main
    loop.  Integer-valued data: bit-exact, the same bits in place and on a second run, also without residual."""
    o = dict(ov, max_ctas=max_ctas, stream_k=3)
    info = kx.kx_plan_query(M, N, K, ov=kx.make_override(**o))
    assert info.stream_k == 2 and info.workspace_bytes > 0 and info.narrow_tiles == 0
    X, W, b, R = ternary_case(M, N, K, seed=25)
    ref = oracle.outproj(X, W, b, R)
    y = run(X, W, b, R, o)
    ok, msg = kt.gate_exact(y, ref)
    assert ok, msg
    assert np.array_equal(run(X, W, b, R.copy(), o, inplace=True), y)
    assert np.array_equal(run(X, W, b, R, o), y)
    ok, msg = kt.gate_exact(run(X, W, None, None, o), oracle.outproj(X, W))
    assert ok, msg
    with pytest.raises(kx.KxError):            # nothing is left over: no region to split
        kx.kx_plan_query(512, 512, 512, ov=kx.make_override(path=T, block_n=256, cta_pair=1, max_ctas=4, stream_k=3))


@pytest.mark.parametrize("ov,max_ctas,M,N,K", [
    (dict(path=T, block_n=256, cta_pair=2), 12, 640, 1280, 520),     # 15 pair tiles on 6 slots: 3 left over, 6 K halves
    (dict(path=T, block_n=256, cta_pair=2, stages=3), 12, 640, 1280, 4096),
    (dict(path=T, block_n=256, cta_pair=1), 10, 640, 1280, 1096),    # 25 tiles on 10 slots: 5 left over, odd k-block count
    (dict(path=T, block_n=128, cta_pair=2), 12, 700, 520, 264),      # ragged rows and columns
    (dict(path=T, block_n=192, cta_pair=1, stages=2), 10, 300, 776, 2048),
    (dict(path=T, block_n=128, cta_pair=1, stages=3), 9, 300, 776, 136),
    (dict(path=T, block_n=256, cta_pair=2), 0, 4096, 2560, 264),     # full grid: 160 pair tiles on 74 slots, 12 left over
], ids=["pair256", "pair256-2kb-longk", "single256", "pair128-ragged", "single192-2kb", "single128-2kb", "pair256-fullgrid"])
def test_k_halves_tail_exact_integer_arithmetic(ov, max_ctas, M, N, K):
    """Tiles left over after the full waves run as two K halves on two slots, which swap through the workspace the
    chunks the other one finishes.  Integer-valued data: bit-exact, the same bits in place and on a second run
    (the flags are back at zero), also without bias and residual."""
    o = dict(ov, max_ctas=max_ctas, narrow_tail=3)
    info = kx.kx_plan_query(M, N, K, ov=kx.make_override(**o))
    assert info.workspace_bytes > 0 and info.narrow_tiles == 0 and info.stream_k == 0
    X, W, b, R = ternary_case(M, N, K, seed=29)
    ref = oracle.outproj(X, W, b, R)
    y = run(X, W, b, R, o)
    ok, msg = kt.gate_exact(y, ref)
    assert ok, msg
    assert np.array_equal(run(X, W, b, R.copy(), o, inplace=True), y)
    assert np.array_equal(run(X, W, b, R, o), y)
    ok, msg = kt.gate_exact(run(X, W, None, None, o), oracle.outproj(X, W))
    assert ok, msg
    with pytest.raises(kx.KxError):            # nothing is left over
        kx.kx_plan_query(512, 512, 512, ov=kx.make_override(path=T, block_n=256, cta_pair=1, max_ctas=4, narrow_tail=3))


def test_tail_choice_follows_the_reduction_length():
    """Automatic plans: tiles left over after the full waves run as K halves from 64 k-blocks on, as half-width
    tiles below, and whole when neither fits; the 8-bit entry points never take K halves."""
    long_k = kx.kx_plan_query(4096, 4096, 4096)
    assert long_k.narrow_tiles == 0 and long_k.workspace_bytes > 0 and long_k.stream_k == 0 and long_k.tiles == 290
    short_k = kx.kx_plan_query(4096, 4096, 2048)
    assert short_k.narrow_tiles == 68 and short_k.workspace_bytes == 0
    none = kx.kx_plan_query(8192, 8192, 8192)                  # 1024 tiles on 74 slots: 62 left over, too many to split
    assert none.narrow_tiles == 0 and none.workspace_bytes == 0 and none.tiles == 1024
    X, W, b, R = ternary_case(1024, 4096, 4096, seed=31)
    y = run(X, W, b, R, None, entry="fused")                   # 64 pair tiles: one wave, nothing left over
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg


@pytest.mark.parametrize("group", [1, 3, 16, 64])
@pytest.mark.parametrize("pair", [1, 2])
def test_raster_group_exact_integer_arithmetic(group, pair):
    """The raster group only reorders tiles: any group size, one larger than the number of tile rows and one that
    does not divide it included, gives the exact result."""
    M, N, K = 1100, 1304, 328
    o = dict(path=T, block_n=128, cta_pair=pair, raster_group=group, max_ctas=8)
    info = kx.kx_plan_query(M, N, K, ov=kx.make_override(**o))
    assert info.raster_group == group
    X, W, b, R = ternary_case(M, N, K, seed=27)
    ok, msg = kt.gate_exact(run(X, W, b, R, o), oracle.outproj(X, W, b, R))
    assert ok, msg


@pytest.mark.parametrize("ov,max_ctas,M,N", [
    (dict(path=T, block_n=256, cta_pair=2), 12, 640, 1280),    # 15 pair tiles on 6 slots: 12 wide + 6 narrow
    (dict(path=T, block_n=256, cta_pair=1), 10, 640, 1280),    # 25 tiles on 10 slots: 20 wide + 10 narrow
    (dict(path=T, block_n=128, cta_pair=2), 12, 700, 520),     # 15 pair tiles on 6 slots, ragged rows and columns
    (dict(path=T, block_n=128, cta_pair=1), 9, 300, 776),
    (dict(path=T, block_n=256, cta_pair=2, stages=3), 12, 640, 1280),     # two k-blocks per ring stage
    (dict(path=T, block_n=128, cta_pair=2, stages=4), 12, 700, 520),
], ids=["pair256", "single256", "pair128-ragged", "single128-ragged", "pair256-2kb", "pair128-2kb-ragged"])
def test_half_width_tail_tiles_exact(ov, max_ctas, M, N):
    """Tiles left over after the full waves run as half-width tiles (second W tensor map,
    narrower MMA, half the epilogue chunks).  Must be bit-exact, also in place."""
    K = 520
    o = dict(ov, max_ctas=max_ctas, narrow_tail=2)
    info = kx.kx_plan_query(M, N, K, ov=kx.make_override(**o))
    assert info.narrow_tiles > 0 and info.narrow_tiles % 2 == 0 and info.stream_k == 0
    X, W, b, R = ternary_case(M, N, K, seed=23)
    ref = oracle.outproj(X, W, b, R)
    y = run(X, W, b, R, o)
    ok, msg = kt.gate_exact(y, ref)
    assert ok, msg
    assert np.array_equal(run(X, W, b, R.copy(), o, inplace=True), y)
    off = dict(ov, max_ctas=max_ctas, narrow_tail=1)
    assert kx.kx_plan_query(M, N, K, ov=kx.make_override(**off)).narrow_tiles == 0
    assert np.array_equal(run(X, W, b, R, off), y)


@pytest.mark.parametrize("bn", [256, 192, 128, 64])
@pytest.mark.parametrize("kc", [2, 4])
@pytest.mark.parametrize("M,N,K", [(128, 256, 512), (512, 2048, 2048), (300, 520, 520), (640, 1032, 4096)])
def test_k_cluster_exact_integer_arithmetic(bn, kc, M, N, K):
    """Single-CTA tiles whose K range is split over a 2- or 4-CTA cluster; the partial tiles are
    summed through distributed shared memory in rank order.  Integer-valued data: bit-exact,
    also in place and without bias / residual."""
    ov = dict(path=T, block_n=bn, cta_pair=1, k_cluster=kc)
    X, W, b, R = ternary_case(M, N, K, seed=27)
    y = run(X, W, b, R, ov)
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg
    assert np.array_equal(run(X, W, b, R.copy(), ov, inplace=True), y)
    ok, msg = kt.gate_exact(run(X, W, None, None, ov), oracle.outproj(X, W))
    assert ok, msg


@pytest.mark.parametrize("bn,stages", [(256, 0), (256, 3), (256, 5), (192, 0), (128, 0), (128, 4)])
@pytest.mark.parametrize("M,N,K", [(256, 256, 512), (512, 2048, 2048), (300, 520, 520), (640, 1032, 4096)])
def test_k_cluster_of_pairs_exact_integer_arithmetic(bn, stages, M, N, K):
    """CTA-pair tiles (256 rows) whose K range is split over two pairs, a cluster of four CTAs; each CTA sums
    the two partials of its 128 rows through distributed shared memory.  Integer-valued data: bit-exact,
    also in place and without bias / residual."""
    ov = dict(path=T, block_n=bn, cta_pair=2, k_cluster=2, stages=stages)
    X, W, b, R = ternary_case(M, N, K, seed=29)
    y = run(X, W, b, R, ov)
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg
    assert np.array_equal(run(X, W, b, R.copy(), ov, inplace=True), y)
    ok, msg = kt.gate_exact(run(X, W, None, None, ov), oracle.outproj(X, W))
    assert ok, msg


def test_k_cluster_of_pairs_is_the_plan_for_a_few_tile_rows():
    info = kx.kx_plan_query(512, 4096, 4096, ov=kx.make_override(no_table=1))
    assert (info.path, info.cta_pair, info.block_n, info.grid, info.tiles) == (T, 2, 256, 128, 32)
    d = inputs.make_inputs(inputs.all_workloads()["sweep_M512_H4096"], stress=True)
    ref, absref = oracle.outproj(d["X"], d["W"], d["bias"], d["R"], want_abs=True)
    ys = [run(d["X"], d["W"], d["bias"], d["R"], dict(no_table=1)) for _ in range(2)]
    assert np.array_equal(ys[0], ys[1])
    ok, msg = kt.gate_a(ys[0], ref)
    assert ok, msg
    ok, msg = kt.gate_c(ys[0], ref, absref, 4096, rate_limit=3e-2)
    assert ok, msg


def test_k_cluster_random_data_and_bad_plans():
    d = inputs.make_inputs(inputs.all_workloads()["sweep_M512_H2048"], stress=True)
    ref, absref = oracle.outproj(d["X"], d["W"], d["bias"], d["R"], want_abs=True)
    for kc in (2, 4):
        ov = dict(path=T, block_n=256, cta_pair=1, k_cluster=kc)
        ys = [run(d["X"], d["W"], d["bias"], d["R"], ov) for _ in range(2)]
        assert np.array_equal(ys[0], ys[1])
        ok, msg = kt.gate_a(ys[0], ref)
        assert ok, msg
        ok, msg = kt.gate_c(ys[0], ref, absref, 2048, rate_limit=3e-2)
        assert ok, msg
    for bad in (dict(path=T, block_n=256, cta_pair=2, k_cluster=4), dict(path=T, block_n=256, cta_pair=1, k_cluster=3),
                dict(path=T, block_n=256, cta_pair=1, k_cluster=2, stream_k=2)):
        with pytest.raises(kx.KxError):
            kx.kx_plan_query(512, 2048, 2048, ov=kx.make_override(**bad))


@pytest.mark.parametrize("depth", [-1, 0, 1, 3, 1000])
@pytest.mark.parametrize("base", [dict(path=T, block_n=256, cta_pair=2), dict(path=T, block_n=128, cta_pair=1),
                                  dict(path=T, block_n=256, cta_pair=1, k_cluster=2), dict(path=T, block_n=256, cta_pair=2, narrow_tail=2),
                                  dict(path=T, block_n=256, cta_pair=2, k_cluster=2),
                                  dict(path=S, block_n=32, split_k=3), dict(path=S, block_n=16, split_k=4, cluster_reduce=2),
                                  dict(path=S, block_n=32, split_k=4, cluster_reduce=3)], ids=vid)
def test_l2_prefetch_depth_changes_no_bit(base, depth):
    """The tiles a CTA requests into L2 ahead of the dependency wait are a hint only: every depth
    (none, ring depth, shallower, deeper than the K range) gives the same bits, and a weight
    matrix rewritten by the previous kernel in the stream is still seen (L2 is coherent)."""
    M, N, K = (600, 776, 1096) if base["path"] == T else (base["block_n"] - 3, 520, 1096)
    X, W, b, R = ternary_case(M, N, K, seed=31)
    y = run(X, W, b, R, dict(base, l2_prefetch=depth))
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg
    # previous kernel in the stream rewrites W: the prefetch may have run before it finished
    import torch
    tX, tR, tb, tW2 = kt.to_dev(X), kt.to_dev(R), kt.to_dev(b), kt.to_dev(W)
    tW = torch.zeros_like(tW2)
    eye = torch.eye(K, dtype=torch.bfloat16, device="cuda")
    tY = kt.nan_filled(M, N)
    ov = kx.make_override(**dict(base, l2_prefetch=depth))
    for _ in range(3):
        tW.zero_()
        kx.kx_gemm_bf16(tW2, eye, tW)      # W = W . I^T, written by the library's own kernel, whose
        kx.kx_outproj_residual_ex(tX, tW, tb, tR, tY, ov)   # tail the next prologue overlaps
    assert np.array_equal(kt.from_dev(tY), y)


@pytest.mark.parametrize("ov", STREAMK_VARIANTS[:2] + [dict(path=T, block_n=256, cta_pair=2, stream_k=3, max_ctas=8)], ids=vid)
def test_stream_k_random_data_is_deterministic_and_within_gates(ov):
    wl = inputs.all_workloads()["cfg2"]
    d = inputs.make_inputs(wl, stress=True, M=1100, N=1304, K=4096)
    ref, absref = oracle.outproj(d["X"], d["W"], None, d["R"], want_abs=True)
    ys = [run(d["X"], d["W"], None, d["R"], ov) for _ in range(3)]
    assert np.array_equal(ys[0], ys[1]) and np.array_equal(ys[0], ys[2])
    ok, msg = kt.gate_a(ys[0], ref)
    assert ok, msg
    ok, msg = kt.gate_c(ys[0], ref, absref, 4096, rate_limit=3e-2)
    assert ok, msg
    # plain GEMM through stream-K
    y = run(d["X"], d["W"], None, None, ov)
    assert kt.rel_fro(y, oracle.outproj(d["X"], d["W"])) <= 2.0 ** -8


@pytest.mark.parametrize("ov", [TILE_VARIANTS[0], TILE_VARIANTS[3], SWAP_VARIANTS[1], SWAP_VARIANTS[6]], ids=vid)
def test_exact_large_k(ov):
    """K = 14336 (the longest reduction of the workloads): any dropped or repeated
    k-block, or a ring-phase slip after many wraps, shows as a bit mismatch."""
    M = 16 if ov["path"] == S and ov["block_n"] == 16 else 256
    X, W, b, R = ternary_case(M, 512, 14336, seed=3)
    y = run(X, W, b, R, ov)
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg


@pytest.mark.parametrize("ov", [None] + TILE_VARIANTS[:1] + TILE_VARIANTS[3:4] + SWAP_VARIANTS[3:4], ids=lambda v: "auto" if v is None else vid(v))
def test_zero_weight_returns_residual_plus_bias(ov):
    """W = 0: Y == R bit for bit without bias; with bias Y == rne(R + bias)."""
    M, N, K = (48 if ov and ov["path"] == S else 384), 520, 320
    d = inputs.make_inputs(inputs.Workload("t", M, N, K, 31, True, True), stress=True)
    W0 = np.zeros((N, K), dtype=np.uint16)
    y = run(d["X"], W0, None, d["R"], ov)
    assert np.array_equal(y, d["R"])
    y = run(d["X"], W0, d["bias"], d["R"], ov)
    f = lambda a: oracle.widen_bf16(a)
    assert np.array_equal(y, oracle.round_bf16(f(d["R"]) + f(d["bias"])[None, :]))


@pytest.mark.parametrize("ov", [TILE_VARIANTS[0], TILE_VARIANTS[2], TILE_VARIANTS[3], SWAP_VARIANTS[2], SWAP_VARIANTS[6],
                                SWAP_VARIANTS[18]], ids=vid)
def test_selectors(ov):
    """W a permutation matrix picks columns of X; one-hot X picks columns of W."""
    M = 24 if ov["path"] == S and ov["block_n"] < 128 else 260
    N, K = 392, 448
    W, pi = inputs.permutation_matrix_bf16(5, N, K)
    X = inputs.normal_bf16(5, "X", (M, K), 1.0)
    y = run(X, W, None, None, ov)
    assert np.array_equal(y, X[:, pi])
    X1 = inputs.one_hot_rows_bf16(M, K)
    Wr = inputs.normal_bf16(6, "W", (N, K), 1.0)
    y = run(X1, Wr, None, None, ov)
    assert np.array_equal(y, Wr[:, np.arange(M) % K].T)


@pytest.mark.parametrize("ov", [TILE_VARIANTS[1], TILE_VARIANTS[3], SWAP_VARIANTS[4]], ids=vid)
def test_power_of_two_scaling_is_bitwise(ov):
    M = 100 if ov["path"] == S else 512
    d = inputs.make_inputs(inputs.Workload("t", M, 512, 1024, 41, False, False), stress=True)
    y1 = run(d["X"], d["W"], None, None, ov)
    X2 = inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(d["X"]))
    y2 = run(X2, d["W"], None, None, ov)
    want = inputs.f32_to_bf16_bits(2.0 * inputs.bf16_bits_to_f32(y1))
    assert np.array_equal(y2, want)


@pytest.mark.parametrize("ov", [None, TILE_VARIANTS[0], TILE_VARIANTS[2], TILE_VARIANTS[3], TILE_VARIANTS[4],
                                SWAP_VARIANTS[1], SWAP_VARIANTS[5], SWAP_VARIANTS[6], SWAP_VARIANTS[18], SWAP_VARIANTS[20]],
                         ids=lambda v: "auto" if v is None else vid(v))
def test_in_place_matches_out_of_place(ov):
    """Y aliased onto R (the paper's destination/residual aliasing) gives the same bits."""
    M = 20 if ov and ov["path"] == S and ov["block_n"] < 128 else 700
    d = inputs.make_inputs(inputs.Workload("t", M, 1032, 512, 51, True, True), stress=True)
    y_out = run(d["X"], d["W"], d["bias"], d["R"], ov)
    y_in = run(d["X"], d["W"], d["bias"], d["R"].copy(), ov, inplace=True)
    assert np.array_equal(y_out, y_in)
    ok, msg = kt.gate_a(y_in, oracle.outproj(d["X"], d["W"], d["bias"], d["R"]))
    assert ok, msg


def test_weight_rewritten_in_place_is_seen():
    """Same pointers, new contents: nothing derived from tensor contents may be cached."""
    M, N, K = 256, 512, 512
    X, W, b, R = ternary_case(M, N, K, seed=7)
    Xd, Wd, bd, Rd = kt.to_dev(X), kt.to_dev(W), kt.to_dev(b), kt.to_dev(R)
    Y = kt.nan_filled(M, N)
    for ov in (None, dict(path=S, block_n=256, split_k=2)):
        o = kx.make_override(**ov) if ov else None
        kx.kx_outproj_residual_ex(Xd, Wd, bd, Rd, Y, o)
        assert kt.gate_exact(kt.from_dev(Y), oracle.outproj(X, W, b, R))[0]
        W2 = inputs.ternary_bf16(8, "W", (N, K))
        Wd.copy_(kt.to_dev(W2))
        kx.kx_outproj_residual_ex(Xd, Wd, bd, Rd, Y, o)
        ok, msg = kt.gate_exact(kt.from_dev(Y), oracle.outproj(X, W2, b, R))
        assert ok, msg
        Wd.copy_(kt.to_dev(W))


def test_repeated_calls_are_deterministic():
    d = inputs.make_inputs(inputs.Workload("t", 77, 2048, 2048, 61, True, True))
    ys = [run(d["X"], d["W"], d["bias"], d["R"], dict(path=S, block_n=128, split_k=8)) for _ in range(3)]
    assert np.array_equal(ys[0], ys[1]) and np.array_equal(ys[0], ys[2])
    d = inputs.make_inputs(inputs.Workload("t", 1024, 1024, 1024, 62, True, True))
    ys = [run(d["X"], d["W"], d["bias"], d["R"]) for _ in range(3)]
    assert np.array_equal(ys[0], ys[1]) and np.array_equal(ys[0], ys[2])


# ------------------------------------------------------------------ tolerance gates on random data
CASES = [
    # (name of recipe, M, N, K) — the workloads' recipes at sizes the oracle finishes in seconds
    ("cfg1", 128, 1024, 1024),      # the small workload at full size
    ("cfg2", 520, 1024, 4096),
    ("cfg5", 384, 512, 14336),
    ("sweep_M1_H2048", 1, 2048, 2048),
    ("sweep_M32_H5120", 32, 5120, 5120),
    ("sweep_M512_H2048", 512, 2048, 2048),
    ("sweep_M8192_H4096", 1100, 1304, 4096),
]


@pytest.mark.parametrize("name,M,N,K", CASES)
@pytest.mark.parametrize("stress", [False, True], ids=["literal", "stress"])
def test_random_workloads_all_gates(name, M, N, K, stress):
    """Gate A (the formal tolerance) and the sharp gate on the workloads' own
    distributions, through the public entry point with the automatic plan.
    `stress` rescales X to N(0,1) so the GEMM term itself is O(1)."""
    wl = inputs.all_workloads()[name]
    d = inputs.make_inputs(wl, stress=stress, M=M, N=N, K=K)
    ref, absref = oracle.outproj(d["X"], d["W"], d["bias"], d["R"], want_abs=True)
    y = run(d["X"], d["W"], d["bias"], d["R"], None, entry="fused")
    ok, msg = kt.gate_a(y, ref)
    assert ok, msg
    ok, msg = kt.gate_c(y, ref, absref, K, rate_limit=3e-2 if stress else 5e-3)
    assert ok, msg


@pytest.mark.parametrize("ov", TILE_VARIANTS + SWAP_VARIANTS[4:], ids=vid)
def test_plain_gemm_relative_error(ov):
    """Plain GEMM on uniform data: relative Frobenius error <= 2^-8 (BF16 rounding
    alone gives ~1.7e-3; a dropped 64-wide k-block would give several percent)."""
    M = 128 if ov["path"] == S and ov["block_n"] == 128 else 600
    wl = inputs.all_workloads()["cfg4"]
    d = inputs.make_inputs(wl, M=M, N=1040, K=2048)
    ref, absref = oracle.outproj(d["X"], d["W"], want_abs=True)
    y = run(d["X"], d["W"], None, None, ov)
    assert kt.rel_fro(y, ref) <= 2.0 ** -8
    ok, msg = kt.gate_c(y, ref, absref, 2048, rate_limit=3e-2)   # no residual: GEMM term is the output
    assert ok, msg
    y2 = run(d["X"], d["W"], None, None, None, entry="gemm")
    assert kt.rel_fro(y2, ref) <= 2.0 ** -8


# ------------------------------------------------------------------ edge cases
@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (1, 8, 64), (3, 16, 8), (129, 8, 72), (257, 264, 8),
                                   (127, 1016, 136), (255, 24, 4096)])
@pytest.mark.parametrize("path", [0, T, S])
def test_small_and_ragged_shapes(M, N, K, path):
    X, W, b, R = ternary_case(M, N, K, seed=9)
    ov = dict(path=path) if path else None
    y = run(X, W, b, R, ov)
    ok, msg = kt.gate_exact(y, oracle.outproj(X, W, b, R))
    assert ok, msg


def test_empty_sum_and_empty_output():
    M, N = 37, 264
    _, _, b, R = ternary_case(M, N, 8, seed=10)
    X0 = np.zeros((M, 0), dtype=np.uint16)
    W0 = np.zeros((N, 0), dtype=np.uint16)
    Rd, bd = kt.to_dev(R), kt.to_dev(b)
    Y = kt.nan_filled(M, N)
    assert kx.kx_outproj_residual(0, 0, bd, Rd, Y, M=M, N=N, K=0) == kx.KX_OK
    f = oracle.widen_bf16
    assert np.array_equal(kt.from_dev(Y), oracle.round_bf16(f(R) + f(b)[None, :]))
    assert np.array_equal(oracle.outproj(X0, W0, b, R), f(R) + f(b)[None, :])
    Y = kt.nan_filled(M, N)
    assert kx.kx_gemm_bf16(0, 0, Y, M=M, N=N, K=0) == kx.KX_OK
    assert not kt.from_dev(Y).any()
    # M == 0 / N == 0: nothing is written, nothing is launched
    Y = kt.nan_filled(4, 8)
    assert kx.kx_gemm_bf16(0, 0, Y, M=0, N=8, K=8) == kx.KX_OK
    assert np.isnan(oracle.widen_bf16(kt.from_dev(Y))).all()


def test_special_values_propagate_only_where_they_should():
    M, N, K = 130, 264, 192
    X, W, b, R = ternary_case(M, N, K, seed=11)
    X = X.copy(); R = R.copy()
    X[5, 70] = 0x7F80          # +inf in one row of X
    X[100, 3] = 0x7FC0         # NaN in another
    R[17, 200] = 0xFF80        # -inf in one residual element
    for ov in (None, dict(path=S, block_n=256, split_k=2)):
        y = oracle.widen_bf16(run(X, W, b, R, ov))
        ref = oracle.outproj(X, W, b, R)
        assert np.array_equal(np.isnan(y), np.isnan(ref))
        fin = np.isfinite(ref)
        assert np.array_equal(y[~np.isnan(ref) & ~fin], ref[~np.isnan(ref) & ~fin])
        assert np.array_equal(oracle.round_bf16(ref[fin]), oracle.round_bf16(y[fin]))
        assert np.isnan(y[100]).all() and y[17, 200] == -np.inf


def test_guard_regions_are_untouched():
    """Canaries before and after Y: the TMA stores and the split-K epilogue must
    not write outside [Y, Y + M*N)."""
    import torch
    M, N, K = 300, 520, 264
    X, W, b, R = ternary_case(M, N, K, seed=12)
    pad = 4096
    for ov in (None, dict(path=T, block_n=256, cta_pair=2), dict(path=S, block_n=256, split_k=3)):
        buf = torch.full((pad + M * N + pad,), -7.0, dtype=torch.bfloat16, device="cuda")
        Y = buf[pad:pad + M * N].view(M, N)
        o = kx.make_override(**ov) if ov else None
        kx.kx_outproj_residual_ex(kt.to_dev(X), kt.to_dev(W), kt.to_dev(b), kt.to_dev(R), Y, o)
        torch.cuda.synchronize()
        assert (buf[:pad] == -7.0).all() and (buf[pad + M * N:] == -7.0).all()
        assert kt.gate_exact(kt.from_dev(Y.contiguous()), oracle.outproj(X, W, b, R))[0]


def test_host_buffer_entry_point():
    import torch
    M, N, K = 200, 520, 1032
    d = inputs.make_inputs(inputs.Workload("t", M, N, K, 71, True, True), stress=True)
    pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
    Xh, Wh, bh, Rh = pin(d["X"]), pin(d["W"]), pin(d["bias"]), pin(d["R"])
    Yh = torch.empty(M, N, dtype=torch.int16).pin_memory()
    kx.kx_outproj_residual_host(Xh, Wh, bh, Rh, Yh, M, N, K)
    y = Yh.numpy().view(np.uint16)
    assert np.array_equal(y, run(d["X"], d["W"], d["bias"], d["R"]))
    ok, msg = kt.gate_a(y, oracle.outproj(d["X"], d["W"], d["bias"], d["R"]))
    assert ok, msg
    # M >= 2048: pipelined row slices; every slice must land in its place (pinned and pageable hosts)
    M3 = 2304 + 77
    d3 = inputs.make_inputs(inputs.Workload("t", M3, 264, 520, 73, True, True), stress=True)
    X3, W3, b3, R3 = ternary_case(M3, 264, 520, seed=74)
    Y3 = torch.empty(M3, 264, dtype=torch.int16).pin_memory()
    kx.kx_outproj_residual_host(pin(X3), pin(W3), pin(b3), pin(R3), Y3, M3, 264, 520)
    ok, msg = kt.gate_exact(Y3.numpy().view(np.uint16), oracle.outproj(X3, W3, b3, R3))
    assert ok, msg
    Y3p = np.zeros((M3, 264), dtype=np.uint16)
    kx.kx_outproj_residual_host(np.ascontiguousarray(d3["X"]), np.ascontiguousarray(d3["W"]), None,
                                np.ascontiguousarray(d3["R"]), Y3p, M3, 264, 520)
    ok, msg = kt.gate_a(Y3p, oracle.outproj(d3["X"], d3["W"], None, d3["R"]))
    assert ok, msg
    # a larger problem afterwards grows the staging buffer
    M2 = 900
    d2 = inputs.make_inputs(inputs.Workload("t", M2, N, K, 72, False, False), stress=True)
    Y2 = np.empty((M2, N), dtype=np.uint16)
    kx.kx_outproj_residual_host(np.ascontiguousarray(d2["X"]), np.ascontiguousarray(d2["W"]), None, None, Y2, M2, N, K)
    assert kt.rel_fro(Y2, oracle.outproj(d2["X"], d2["W"])) <= 2.0 ** -8


def test_non_default_stream_and_plan_query():
    import torch
    info = kx.kx_plan_query(4096, 4096, 4096)
    assert info.path == T and info.grid >= 1 and info.launches == 1 and info.tiles >= info.grid // 2
    info = kx.kx_plan_query(32, 8192, 8192)
    assert info.path == S and info.block_n == 32 and info.split_k >= 1
    ws = info.split_k * 32 * 8192 * 4 if (info.split_k > 1 and not info.cluster_reduce) else 0
    assert info.workspace_bytes == ws and (info.cluster_reduce == 0 or 2 <= info.split_k <= 8)
    assert info.cluster_reduce == 1          # the splits form a cluster; finishers pull the partial rows
    assert kx.kx_plan_query(32, 8192, 8192, ov=kx.make_override(path=S, cluster_reduce=3)).cluster_reduce == 2
    with pytest.raises(kx.KxError):          # no push form with 256 rows of X per unit
        kx.kx_plan_query(200, 4096, 4096, ov=kx.make_override(path=S, block_n=256, split_k=2, cluster_reduce=3))
    with pytest.raises(kx.KxError):
        kx.kx_plan_query(4096, 4096, 4096, ov=kx.make_override(path=T, block_n=96))
    X, W, b, R = ternary_case(256, 512, 256, seed=13)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        y = run(X, W, b, R)
    assert kt.gate_exact(y, oracle.outproj(X, W, b, R))[0]
