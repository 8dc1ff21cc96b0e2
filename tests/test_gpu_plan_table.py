"""The measured plan table: a listed shape takes its table plan (and still matches the
oracle), `no_table` or any explicit plan field bypasses it, and shapes that are not
listed fall back to the heuristic."""
import os
import re

import numpy as np
import pytest

import oracle
from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import inputs

import kxtest as kt

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FIELDS = ("path", "block_n", "cta_pair", "split_k", "raster_group", "stages", "stream_k", "narrow_tail",
          "cluster_reduce", "k_cluster")


def table_entries():
    text = open(os.path.join(ROOT, "paper_2608_17071_b200", "csrc", "kx_plan_table.inc")).read()
    out = []
    for line in text.splitlines():
        m = re.match(r"\s*\{([^}]*)\}", line)
        if m:
            v = [int(x) for x in m.group(1).split(",")]
            out.append(dict(m_lo=v[0], m_hi=v[1], N=v[2], K=v[3], **dict(zip(FIELDS, v[4:]))))
    return out


def test_table_entries_are_used_and_correct():
    for e in table_entries():
        for M in sorted({e["m_lo"], e["m_hi"]}):
            info = kx.kx_plan_query(M, e["N"], e["K"])
            assert info.from_table == 1
            assert info.path == e["path"] and info.block_n == e["block_n"]
            if e["split_k"]:
                assert info.split_k == min(e["split_k"], (e["K"] + 63) // 64)
            heur = kx.kx_plan_query(M, e["N"], e["K"], ov=kx.make_override(no_table=1))
            assert heur.from_table == 0
            # an explicit plan field also bypasses the table
            pinned = kx.kx_plan_query(M, e["N"], e["K"], ov=kx.make_override(path=kx.KX_PATH_TILE, block_n=64))
            assert pinned.from_table == 0 and pinned.block_n == 64
            # the table plan reproduces the oracle bit for bit on exact-arithmetic inputs
            X = inputs.ternary_bf16(31, "X", (M, e["K"]))
            W = inputs.ternary_bf16(31, "W", (e["N"], e["K"]))
            b = inputs.small_int_bf16(31, "bias", (e["N"],), -4, 4)
            R = inputs.small_int_bf16(31, "R", (M, e["N"]), -8, 8)
            Y = kt.nan_filled(M, e["N"])
            kx.kx_outproj_residual(kt.to_dev(X), kt.to_dev(W), kt.to_dev(b), kt.to_dev(R), Y)
            assert kx.kx_last_device_status()[0] == kx.KX_OK
            ok, msg = kt.gate_exact(kt.from_dev(Y), oracle.outproj(X, W, b, R))
            assert ok, msg


def test_unlisted_shapes_fall_back_to_the_heuristic():
    listed = {(e["N"], e["K"]) for e in table_entries()}
    for (M, N, K) in [(100, 1032, 1024), (4096, 4096, 4096), (3, 520, 264)]:
        if (N, K) in listed:
            continue
        assert kx.kx_plan_query(M, N, K).from_table == 0
    # same (N, K) as an entry but M outside its bucket
    for e in table_entries():
        assert kx.kx_plan_query(e["m_hi"] + 1, e["N"], e["K"]).from_table == 0
