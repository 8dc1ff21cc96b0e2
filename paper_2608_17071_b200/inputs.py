"""Seeded synthetic inputs for the BF16 output projection with residual.

This module is the ONLY thing the CPU oracle's tests and the CUDA path share.
It holds no arithmetic of the method itself (no products, no sums, no output
rounding): it only draws numbers and packs them as BF16 bit patterns
(``numpy.uint16``), which both sides then consume unchanged.

Generator: numpy's counter-based Philox bit generator keyed on
``(seed, tensor_id)`` with tensor ids X=0, W=1, bias=2, R=3, so each tensor of
each workload is an independent, reproducible stream regardless of the order
in which tensors are requested.  Values are drawn in FP32, scaled in FP32 and
rounded to BF16 with round-to-nearest-even.

Workloads (the five synthetic configurations the project is measured on):

* ``cfg1``  out-proj + bias + residual, M=128,  K=N=1024, seed 0
* ``cfg2``  out-proj + residual (no bias), M=K=N=4096, seed 1
* ``sweep`` 16 shapes, M in {1,32,512,8192} x hidden K=N in
  {2048,4096,5120,8192}, with bias; seed 2+i, i = 4*iM + iH (M outer)
* ``cfg4``  plain GEMM M=N=K=8192, X,W ~ U(-1,1)/sqrt(K), seed 20
* ``cfg5``  M=16384, K=14336, N=4096, with bias, seed 21

X and W are N(0,1)/sqrt(K) (both operands scaled: the literal reading of the
workload text), R ~ N(0,1), bias ~ N(0,0.1).  ``stress=True`` gives the
parity-only variant with X ~ N(0,1) so that the GEMM term itself is O(1).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np

TENSOR_ID = {"X": 0, "W": 1, "bias": 2, "R": 3}

SWEEP_M = (1, 32, 512, 8192)
SWEEP_H = (2048, 4096, 5120, 8192)


# --------------------------------------------------------------------------
# BF16 packing (input production only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round an FP32 array to BF16 (round-to-nearest-even), return uint16 bits."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + (np.uint32(0x7FFF) + lsb)
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen BF16 bit patterns to FP32 (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, tensor: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), TENSOR_ID[tensor]]))


_CHUNK = 1 << 24


def normal_bf16(seed: int, tensor: str, shape, std: float) -> np.ndarray:
    """N(0, std^2) in FP32, rounded to BF16 bits.  Drawn in fixed-size chunks of
    the flattened tensor so memory stays bounded for the largest operands."""
    n = int(np.prod(shape))
    g = _rng(seed, tensor)
    out = np.empty(n, dtype=np.uint16)
    s = np.float32(std)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        v = g.standard_normal(hi - lo, dtype=np.float32)
        v *= s
        out[lo:hi] = f32_to_bf16_bits(v)
    return out.reshape(shape)


def uniform_bf16(seed: int, tensor: str, shape, half_width: float) -> np.ndarray:
    """U(-half_width, half_width) in FP32, rounded to BF16 bits."""
    n = int(np.prod(shape))
    g = _rng(seed, tensor)
    out = np.empty(n, dtype=np.uint16)
    w = np.float32(half_width)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        v = g.random(hi - lo, dtype=np.float32)
        v = (v * np.float32(2.0) - np.float32(1.0)) * w
        out[lo:hi] = f32_to_bf16_bits(v)
    return out.reshape(shape)


# --------------------------------------------------------------------------
# Workload descriptions
# --------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    M: int
    N: int
    K: int
    seed: int
    has_bias: bool
    has_residual: bool
    dist: str = "normal"  # "normal" | "uniform"

    @property
    def flops(self) -> float:
        return 2.0 * self.M * self.N * self.K

    @property
    def algorithmic_bytes(self) -> float:
        """Each operand read once, Y written once (BF16 = 2 bytes)."""
        b = 2.0 * (self.M * self.K + self.N * self.K + self.M * self.N)
        if self.has_residual:
            b += 2.0 * self.M * self.N
        if self.has_bias:
            b += 2.0 * self.N
        return b


def sweep_workloads() -> List[Workload]:
    out = []
    for im, m in enumerate(SWEEP_M):
        for ih, h in enumerate(SWEEP_H):
            i = 4 * im + ih
            out.append(Workload(f"sweep_M{m}_H{h}", m, h, h, 2 + i, True, True))
    return out


def all_workloads() -> Dict[str, Workload]:
    w = {
        "cfg1": Workload("cfg1", 128, 1024, 1024, 0, True, True),
        "cfg2": Workload("cfg2", 4096, 4096, 4096, 1, False, True),
        "cfg4": Workload("cfg4", 8192, 8192, 8192, 20, False, False, "uniform"),
        "cfg5": Workload("cfg5", 16384, 4096, 14336, 21, True, True),
        # context only: the shape of the paper's fixed-shape GEMM study
        "gemm4096": Workload("gemm4096", 4096, 4096, 4096, 22, False, False, "uniform"),
    }
    for s in sweep_workloads():
        w[s.name] = s
    return w


def make_inputs(wl: Workload, stress: bool = False,
                M: Optional[int] = None, N: Optional[int] = None,
                K: Optional[int] = None) -> Dict[str, Optional[np.ndarray]]:
    """BF16 bit arrays for a workload.  M/N/K override the shape (same recipe,
    same seed) for reduced-size parity cases."""
    M = wl.M if M is None else M
    N = wl.N if N is None else N
    K = wl.K if K is None else K
    inv = 1.0 / math.sqrt(K)
    if wl.dist == "uniform":
        X = uniform_bf16(wl.seed, "X", (M, K), inv)
        W = uniform_bf16(wl.seed, "W", (N, K), inv)
    else:
        X = normal_bf16(wl.seed, "X", (M, K), 1.0 if stress else inv)
        W = normal_bf16(wl.seed, "W", (N, K), inv)
    bias = normal_bf16(wl.seed, "bias", (N,), 0.1) if wl.has_bias else None
    R = normal_bf16(wl.seed, "R", (M, N), 1.0) if wl.has_residual else None
    return {"X": X, "W": W, "bias": bias, "R": R, "M": M, "N": N, "K": K}


# --------------------------------------------------------------------------
# Structured inputs for exact (bit-for-bit) pins.  Still only data.
# --------------------------------------------------------------------------
def ternary_bf16(seed: int, tensor: str, shape) -> np.ndarray:
    """iid values in {-1, 0, +1} as BF16 bits (all exactly representable)."""
    g = _rng(seed, tensor)
    v = g.integers(-1, 2, size=shape, dtype=np.int8).astype(np.float32)
    return f32_to_bf16_bits(v).reshape(shape)


def small_int_bf16(seed: int, tensor: str, shape, lo: int = -8, hi: int = 8) -> np.ndarray:
    """iid integers in [lo, hi] as BF16 bits (exactly representable for |v| <= 256)."""
    g = _rng(seed, tensor)
    v = g.integers(lo, hi + 1, size=shape, dtype=np.int16).astype(np.float32)
    return f32_to_bf16_bits(v).reshape(shape)


def permutation_matrix_bf16(seed: int, n: int, k: int):
    """W[n_, k_] = 1 iff k_ == pi(n_) with pi a seeded map [0,n) -> [0,k);
    returns (bits, pi)."""
    g = _rng(seed, "W")
    if n <= k:
        pi = g.permutation(k)[:n]
    else:
        pi = g.integers(0, k, size=n)
    W = np.zeros((n, k), dtype=np.uint16)
    W[np.arange(n), pi] = np.uint16(0x3F80)  # 1.0
    return W, pi.astype(np.int64)


def one_hot_rows_bf16(m: int, k: int) -> np.ndarray:
    """X[m_, k_] = 1 iff k_ == m_ mod k."""
    X = np.zeros((m, k), dtype=np.uint16)
    X[np.arange(m), np.arange(m) % k] = np.uint16(0x3F80)
    return X


def sampled_rows(M: int, tile: int = 128) -> np.ndarray:
    """Deterministic stratified row sample: two rows per `tile`-row block at
    offsets (37 t + 61 j) mod tile, plus rows 0 and M-1."""
    rows = {0, M - 1}
    for t in range((M + tile - 1) // tile):
        for j in range(2):
            r = t * tile + (37 * t + 61 * j) % tile
            if r < M:
                rows.add(r)
    return np.array(sorted(rows), dtype=np.int64)
