"""The N > 1 path of the benchmark on CPU (gloo, world size 2): rows shard with
no exchange, the step time is the max over ranks, and under the reference arm
only rank 0 works and prints."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import oracle
    from paper_2608_17071_b200 import inputs
    wl = inputs.Workload("t", 48, 64, 96, 5, True, True)
    bits = bench.shard_inputs(inputs, wl, rank)
    ref = oracle.outproj(bits["X"], bits["W"], bits["bias"], bits["R"])
    np.save(os.path.join(out_dir, f"ref{rank}.npy"), ref)
    for k in ("X", "W", "bias", "R"):
        np.save(os.path.join(out_dir, f"{k}{rank}.npy"), bits[k])
    t = bench.max_over_ranks(dist, 1.0 + rank, "cpu")
    assert t == float(world), t
    dist.barrier()
    dist.destroy_process_group()


def test_row_shards_need_no_exchange(tmp_path):
    import oracle
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    ld = lambda k, r: np.load(tmp_path / f"{k}{r}.npy")
    # W and bias are replicated, X and R differ per rank
    assert np.array_equal(ld("W", 0), ld("W", 1)) and np.array_equal(ld("bias", 0), ld("bias", 1))
    assert not np.array_equal(ld("X", 0), ld("X", 1)) and not np.array_equal(ld("R", 0), ld("R", 1))
    # the stacked problem's reference is the stack of the per-rank references
    X = np.concatenate([ld("X", 0), ld("X", 1)])
    R = np.concatenate([ld("R", 0), ld("R", 1)])
    whole = oracle.outproj(X, ld("W", 0), ld("bias", 0), R)
    assert np.array_equal(whole, np.concatenate([ld("ref", 0), ld("ref", 1)]))


def test_reference_arm_two_ranks_prints_once():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"]
    p = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "bf16_tflops" and d["n_gpus"] == 2
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0


def test_bench_roofline_arithmetic():
    import bench
    from paper_2608_17071_b200 import inputs
    peaks = {"hbm_gbs": 6000.0, "bf16_tflops": 1500.0, "bf16_tflops_sustained": 1200.0, "source": "measured"}
    wl = inputs.all_workloads()["cfg2"]
    r = bench.roof(wl, wl.flops / 750e12, peaks, False)
    assert r["bound"] == "tensor" and abs(r["frac"] - 0.5) < 1e-12 and r["peak"] == 1500.0
    assert bench.roof(wl, 1e-4, peaks, True)["peak"] == 1200.0
    wl = inputs.all_workloads()["sweep_M1_H8192"]
    r = bench.roof(wl, wl.algorithmic_bytes / 3000e9, peaks, False)
    assert r["bound"] == "hbm" and abs(r["frac"] - 0.5) < 1e-12 and r["unit"] == "GB/s"
    assert bench.sets_needed(inputs.all_workloads()["cfg2"]) == 2
    assert bench.sets_needed(inputs.all_workloads()["sweep_M1_H2048"]) == 24
