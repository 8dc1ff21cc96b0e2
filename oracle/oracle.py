"""ctypes wrapper around the plain-C oracle (test infrastructure, CPU only).

All tensors are numpy ``uint16`` arrays holding BF16 bit patterns, row-major:
X [M,K], W [N,K], bias [N] or None, R [M,N] or None.  Results are unrounded
float64.  The definition implemented is the paper's residual GEMM epilogue
(Appendix A, Algorithm 3: O <- W^T A + O with alpha = beta = 1) in row-major
form, plus an optional bias; with bias = R = None it is the plain product of
the paper's fixed-shape GEMM study (Section 4.1).
"""
from __future__ import annotations

import ctypes
from typing import Optional, Tuple

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        p = ctypes.c_void_p
        i64 = ctypes.c_int64
        lib.kx_oracle_outproj_rows.argtypes = [p, p, p, p, p, i64, p, p, i64, i64, i64, ctypes.c_int]
        lib.kx_oracle_outproj_rows.restype = ctypes.c_int
        lib.kx_oracle_element.argtypes = [p, p, p, p, i64, i64, i64, i64]
        lib.kx_oracle_element.restype = ctypes.c_double
        lib.kx_oracle_round_bf16.argtypes = [p, p, i64]
        lib.kx_oracle_round_bf16.restype = None
        lib.kx_oracle_widen_bf16.argtypes = [p, p, i64]
        lib.kx_oracle_widen_bf16.restype = None
        lib.kx_oracle_rmsnorm_rows.argtypes = [p, p, ctypes.c_double, p, i64, p, i64, i64]
        lib.kx_oracle_rmsnorm_rows.restype = ctypes.c_int
        lib.kx_oracle_swiglu_rows.argtypes = [p, p, p, p, i64, p, p, p, i64, i64, i64]
        lib.kx_oracle_swiglu_rows.restype = ctypes.c_int
        lib.kx_oracle_quantize_rows.argtypes = [p, i64, i64, p, p]
        lib.kx_oracle_swiglu_int8_rows.argtypes = [p, p, p, p, p, p, p, i64, p, p, p, i64, i64, i64]
        lib.kx_oracle_outproj_int8_rows.argtypes = [p, p, p, p, p, p, p, i64, p, i64, i64, i64]
        lib.kx_oracle_e4m3_decode.argtypes = [p, p, i64]
        lib.kx_oracle_e4m3_encode.argtypes = [p, p, i64]
        lib.kx_oracle_quantize_rows_fp8.argtypes = [p, i64, i64, p, p]
        lib.kx_oracle_swiglu_fp8_rows.argtypes = [p, p, p, p, p, p, p, i64, p, i64, i64, i64]
        lib.kx_oracle_outproj_fp8_rows.argtypes = [p, p, p, p, p, p, p, i64, p, i64, i64, i64]
        lib.kx_oracle_e8m0_decode.argtypes = [p, p, i64]
        lib.kx_oracle_quantize_rows_mx.argtypes = [p, i64, i64, p, p]
        lib.kx_oracle_outproj_mx_rows.argtypes = [p, p, p, p, p, p, p, i64, p, i64, i64, i64]
        lib.kx_oracle_e2m1_decode.argtypes = [p, p, i64]
        lib.kx_oracle_e2m1_encode.argtypes = [p, p, i64]
        lib.kx_oracle_quantize_rows_nvfp4.argtypes = [p, i64, i64, ctypes.c_float, p, p]
        lib.kx_oracle_outproj_nvfp4_rows.argtypes = [p, p, p, p, ctypes.c_double, p, p, p, i64, p, i64, i64, i64]
        lib.kx_oracle_max_threads.argtypes = []
        lib.kx_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _bits(a: Optional[np.ndarray], shape, name: str) -> Optional[np.ndarray]:
    if a is None:
        return None
    if a.dtype != np.uint16:
        raise TypeError(f"{name} must be uint16 BF16 bits, got {a.dtype}")
    if tuple(a.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {a.shape}, expected {tuple(shape)}")
    return np.ascontiguousarray(a)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def max_threads() -> int:
    return int(_load().kx_oracle_max_threads())


def outproj_rows(X, W, bias, R, rows, want_abs: bool = False, threads: int = 0
                 ) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """Reference for the given rows (None = all rows): returns (ref, absref)."""
    lib = _load()
    M, K = X.shape
    N = W.shape[0]
    X = _bits(X, (M, K), "X")
    W = _bits(W, (N, K), "W")
    bias = _bits(bias, (N,), "bias")
    R = _bits(R, (M, N), "R")
    if rows is None:
        rows_arr = None
        nrows = M
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        nrows = int(rows_arr.size)
    ref = np.empty((nrows, N), dtype=np.float64)
    absref = np.empty((nrows, N), dtype=np.float64) if want_abs else None
    rc = lib.kx_oracle_outproj_rows(_ptr(X), _ptr(W), _ptr(bias), _ptr(R), _ptr(rows_arr), nrows,
                                    _ptr(ref), _ptr(absref), M, N, K, int(threads))
    if rc != 0:
        raise RuntimeError(f"kx_oracle_outproj_rows failed ({rc})")
    return ref, absref


def outproj(X, W, bias=None, R=None, want_abs: bool = False, threads: int = 0):
    """Reference for the whole output: ref[M,N] float64 (and absref if asked)."""
    ref, absref = outproj_rows(X, W, bias, R, None, want_abs, threads)
    return (ref, absref) if want_abs else ref


def element(X, W, bias, R, m: int, n: int) -> float:
    """Reference for one output element."""
    lib = _load()
    M, K = X.shape
    N = W.shape[0]
    X = _bits(X, (M, K), "X")
    W = _bits(W, (N, K), "W")
    bias = _bits(bias, (N,), "bias")
    R = _bits(R, (M, N), "R")
    if not (0 <= m < M and 0 <= n < N):
        raise IndexError((m, n))
    return float(lib.kx_oracle_element(_ptr(X), _ptr(W), _ptr(bias), _ptr(R), m, n, N, K))


def round_bf16(a: np.ndarray) -> np.ndarray:
    """float64 -> BF16 bits with a single round-to-nearest-even."""
    a = np.ascontiguousarray(a, dtype=np.float64)
    out = np.empty(a.shape, dtype=np.uint16)
    _load().kx_oracle_round_bf16(_ptr(a), _ptr(out), a.size)
    return out


def widen_bf16(bits: np.ndarray) -> np.ndarray:
    """BF16 bits -> float64 (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().kx_oracle_widen_bf16(_ptr(bits), _ptr(out), bits.size)
    return out


def rmsnorm(H, gamma, eps: float, rows=None) -> np.ndarray:
    """RMSNorm of rows of a BF16 matrix: z = h / sqrt(mean_j h_j^2 + eps) * gamma, float64,
    unrounded (textbook definition; the step after the output projection in the paper's
    decoder-layer case study, Appendix A, Algorithm 7).  H [M,N] and gamma [N] are uint16
    BF16 bit patterns; `rows` selects rows (None = all)."""
    lib = _load()
    M, N = H.shape
    H = _bits(H, (M, N), "H")
    gamma = _bits(gamma, (N,), "gamma")
    if rows is None:
        rows_arr, nrows = None, M
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        nrows = int(rows_arr.size)
    out = np.empty((nrows, N), dtype=np.float64)
    rc = lib.kx_oracle_rmsnorm_rows(_ptr(H), _ptr(gamma), float(eps), _ptr(rows_arr), nrows, _ptr(out), M, N)
    if rc != 0:
        raise RuntimeError(f"kx_oracle_rmsnorm_rows failed ({rc})")
    return out


def swiglu(X, Wg, Wu, rows=None, want_parts: bool = False):
    """z = silu(X Wg^T) * (X Wu^T) in float64, unrounded (gate/up projections with the SwiGLU
    product, Appendix A, Algorithm 7 of the paper).  X [M,K], Wg / Wu [I,K] uint16 BF16 bits.
    `rows` selects rows of X; with `want_parts` also returns the gate and up pre-activations."""
    lib = _load()
    M, K = X.shape
    I = Wg.shape[0]
    X = _bits(X, (M, K), "X")
    Wg = _bits(Wg, (I, K), "Wg")
    Wu = _bits(Wu, (I, K), "Wu")
    if rows is None:
        rows_arr, nrows = None, M
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        nrows = int(rows_arr.size)
    out = np.empty((nrows, I), dtype=np.float64)
    g = np.empty((nrows, I), dtype=np.float64) if want_parts else None
    u = np.empty((nrows, I), dtype=np.float64) if want_parts else None
    rc = lib.kx_oracle_swiglu_rows(_ptr(X), _ptr(Wg), _ptr(Wu), _ptr(rows_arr), nrows, _ptr(out), _ptr(g), _ptr(u),
                                   M, I, K)
    if rc != 0:
        raise RuntimeError(f"kx_oracle_swiglu_rows failed ({rc})")
    return (out, g, u) if want_parts else out



def _rows_arg(rows, M):
    if rows is None:
        return None, M
    arr = np.ascontiguousarray(rows, dtype=np.int64)
    return arr, int(arr.size)


def _typed(a, dtype, shape, name):
    a = np.ascontiguousarray(a)
    if a.dtype != dtype or a.shape != tuple(shape):
        raise ValueError(f"{name}: expected {np.dtype(dtype).name}{tuple(shape)}, got {a.dtype}{a.shape}")
    return a


def quantize_rows(Z):
    """Symmetric per-row INT8 code book of BF16 rows (the activation / weight quantisation steps of
    Appendix A, Algorithm 7): scale = max|z| / 127, q = clamp(rint(z * (127 / max|z|))), every
    operation in binary32 (a zero row gets scale 1 and codes 0).  Z [rows, cols] uint16 BF16 bits
    -> (Q int8 [rows, cols], S float32 [rows])."""
    rows, cols = Z.shape
    Z = _bits(Z, (rows, cols), "Z")
    Q = np.empty((rows, cols), dtype=np.int8)
    S = np.empty((rows,), dtype=np.float32)
    rc = _load().kx_oracle_quantize_rows(_ptr(Z), rows, cols, _ptr(Q), _ptr(S))
    if rc != 0:
        raise RuntimeError(f"kx_oracle_quantize_rows failed ({rc})")
    return Q, S


def swiglu_int8(Xq, sx, Wgq, sg, Wuq, su, rows=None, want_acc: bool = False):
    """z = silu(g) * u with g = (Xq Wgq^T) sx sg, u = (Xq Wuq^T) sx su: exact integer sums,
    dequantised and combined in float64, unrounded (INT8 gate/up GEMM with fused dequantisation
    and SwiGLU epilogue, Appendix A, Algorithm 7).  With `want_acc` also the two int64 sums."""
    M, K = Xq.shape
    I = Wgq.shape[0]
    Xq = _typed(Xq, np.int8, (M, K), "Xq")
    Wgq = _typed(Wgq, np.int8, (I, K), "Wgq")
    Wuq = _typed(Wuq, np.int8, (I, K), "Wuq")
    sx = _typed(sx, np.float32, (M,), "sx")
    sg = _typed(sg, np.float32, (I,), "sg")
    su = _typed(su, np.float32, (I,), "su")
    rows_arr, nrows = _rows_arg(rows, M)
    out = np.empty((nrows, I), dtype=np.float64)
    ga = np.empty((nrows, I), dtype=np.int64) if want_acc else None
    ua = np.empty((nrows, I), dtype=np.int64) if want_acc else None
    rc = _load().kx_oracle_swiglu_int8_rows(_ptr(Xq), _ptr(sx), _ptr(Wgq), _ptr(sg), _ptr(Wuq), _ptr(su),
                                            _ptr(rows_arr), nrows, _ptr(out), _ptr(ga), _ptr(ua), M, I, K)
    if rc != 0:
        raise RuntimeError(f"kx_oracle_swiglu_int8_rows failed ({rc})")
    return (out, ga, ua) if want_acc else out


def outproj_int8(Xq, sx, Wq, sw, bias=None, R=None, rows=None):
    """y = (Xq Wq^T) sx sw + bias + R: exact integer sum, the rest in float64, unrounded (the
    output projection with residual of Appendix A, Algorithm 3, on INT8 codes)."""
    M, K = Xq.shape
    N = Wq.shape[0]
    Xq = _typed(Xq, np.int8, (M, K), "Xq")
    Wq = _typed(Wq, np.int8, (N, K), "Wq")
    sx = _typed(sx, np.float32, (M,), "sx")
    sw = _typed(sw, np.float32, (N,), "sw")
    bias = _bits(bias, (N,), "bias")
    R = _bits(R, (M, N), "R")
    rows_arr, nrows = _rows_arg(rows, M)
    out = np.empty((nrows, N), dtype=np.float64)
    rc = _load().kx_oracle_outproj_int8_rows(_ptr(Xq), _ptr(sx), _ptr(Wq), _ptr(sw), _ptr(bias), _ptr(R),
                                             _ptr(rows_arr), nrows, _ptr(out), M, N, K)
    if rc != 0:
        raise RuntimeError(f"kx_oracle_outproj_int8_rows failed ({rc})")
    return out


def e4m3_decode(codes) -> np.ndarray:
    """FP8 E4M3 (bias 7, no infinities, 0x7F / 0xFF NaN, max 448) bit patterns -> float64, exact."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(codes.shape, dtype=np.float64)
    _load().kx_oracle_e4m3_decode(_ptr(codes), _ptr(out), codes.size)
    return out


def e4m3_encode(x) -> np.ndarray:
    """binary32 -> nearest E4M3 code, ties to even, saturating to +-448, NaN -> 0x7F."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint8)
    _load().kx_oracle_e4m3_encode(_ptr(x), _ptr(out), x.size)
    return out


def quantize_rows_fp8(Z):
    """Per-row FP8 code book of BF16 rows: scale = max|z| / 448, q = e4m3(z * (448 / max|z|)), in
    binary32 (the other low-precision operand type of the paper's precision axis, Section 3.2).
    Z uint16 BF16 bits -> (Q uint8 E4M3 bits, S float32)."""
    rows, cols = Z.shape
    Z = _bits(Z, (rows, cols), "Z")
    Q = np.empty((rows, cols), dtype=np.uint8)
    S = np.empty((rows,), dtype=np.float32)
    rc = _load().kx_oracle_quantize_rows_fp8(_ptr(Z), rows, cols, _ptr(Q), _ptr(S))
    if rc != 0:
        raise RuntimeError(f"kx_oracle_quantize_rows_fp8 failed ({rc})")
    return Q, S


def swiglu_fp8(Xq, sx, Wgq, sg, Wuq, su, rows=None):
    """z = silu(g) * u on E4M3 codes, g = (Xq Wgq^T) sx sg, u = (Xq Wuq^T) sx su; float64, unrounded."""
    M, K = Xq.shape
    I = Wgq.shape[0]
    Xq = _typed(Xq, np.uint8, (M, K), "Xq")
    Wgq = _typed(Wgq, np.uint8, (I, K), "Wgq")
    Wuq = _typed(Wuq, np.uint8, (I, K), "Wuq")
    sx = _typed(sx, np.float32, (M,), "sx")
    sg = _typed(sg, np.float32, (I,), "sg")
    su = _typed(su, np.float32, (I,), "su")
    rows_arr, nrows = _rows_arg(rows, M)
    out = np.empty((nrows, I), dtype=np.float64)
    rc = _load().kx_oracle_swiglu_fp8_rows(_ptr(Xq), _ptr(sx), _ptr(Wgq), _ptr(sg), _ptr(Wuq), _ptr(su),
                                           _ptr(rows_arr), nrows, _ptr(out), M, I, K)
    if rc != 0:
        raise RuntimeError(f"kx_oracle_swiglu_fp8_rows failed ({rc})")
    return out


def outproj_fp8(Xq, sx, Wq, sw, bias=None, R=None, rows=None):
    """y = (Xq Wq^T) sx sw + bias + R on E4M3 codes; float64, unrounded."""
    M, K = Xq.shape
    N = Wq.shape[0]
    Xq = _typed(Xq, np.uint8, (M, K), "Xq")
    Wq = _typed(Wq, np.uint8, (N, K), "Wq")
    sx = _typed(sx, np.float32, (M,), "sx")
    sw = _typed(sw, np.float32, (N,), "sw")
    bias = _bits(bias, (N,), "bias")
    R = _bits(R, (M, N), "R")
    rows_arr, nrows = _rows_arg(rows, M)
    out = np.empty((nrows, N), dtype=np.float64)
    rc = _load().kx_oracle_outproj_fp8_rows(_ptr(Xq), _ptr(sx), _ptr(Wq), _ptr(sw), _ptr(bias), _ptr(R),
                                            _ptr(rows_arr), nrows, _ptr(out), M, N, K)
    if rc != 0:
        raise RuntimeError(f"kx_oracle_outproj_fp8_rows failed ({rc})")
    return out


def e8m0_decode(e) -> np.ndarray:
    """E8M0 scale bytes -> float64: 2^(e - 127), 0xFF = NaN."""
    e = np.ascontiguousarray(e, dtype=np.uint8)
    out = np.empty(e.shape, dtype=np.float64)
    _load().kx_oracle_e8m0_decode(_ptr(e), _ptr(out), e.size)
    return out


def quantize_rows_mx(Z):
    """Block-scaled FP8 code book of BF16 rows (Section 3.2, precision axis): per 32 consecutive elements
    one E8M0 scale byte e = clamp(floor(log2 max|z|) - 8 + 127, 0, 254) (zero block: 127) and
    q = e4m3(z / 2^(e-127)).  Z uint16 BF16 bits [rows, cols] -> (Q uint8 [rows, cols],
    E uint8 [rows, ceil(cols / 32)])."""
    rows, cols = Z.shape
    Z = _bits(Z, (rows, cols), "Z")
    Q = np.empty((rows, cols), dtype=np.uint8)
    E = np.empty((rows, (cols + 31) // 32), dtype=np.uint8)
    rc = _load().kx_oracle_quantize_rows_mx(_ptr(Z), rows, cols, _ptr(Q), _ptr(E))
    if rc != 0:
        raise RuntimeError(f"kx_oracle_quantize_rows_mx failed ({rc})")
    return Q, E


def outproj_mx(Xq, ex, Wq, ew, bias=None, R=None, rows=None):
    """y = sum_j 2^(ex[m,j]-127) 2^(ew[n,j]-127) (Xq[m, 32j:32j+32] . Wq[n, 32j:32j+32]) + bias + R on E4M3
    codes with E8M0 block scales; float64, unrounded."""
    M, K = Xq.shape
    N = Wq.shape[0]
    nb = (K + 31) // 32
    Xq = _typed(Xq, np.uint8, (M, K), "Xq")
    Wq = _typed(Wq, np.uint8, (N, K), "Wq")
    ex = _typed(ex, np.uint8, (M, nb), "ex")
    ew = _typed(ew, np.uint8, (N, nb), "ew")
    bias = _bits(bias, (N,), "bias")
    R = _bits(R, (M, N), "R")
    rows_arr, nrows = _rows_arg(rows, M)
    out = np.empty((nrows, N), dtype=np.float64)
    rc = _load().kx_oracle_outproj_mx_rows(_ptr(Xq), _ptr(ex), _ptr(Wq), _ptr(ew), _ptr(bias), _ptr(R),
                                           _ptr(rows_arr), nrows, _ptr(out), M, N, K)
    if rc != 0:
        raise RuntimeError(f"kx_oracle_outproj_mx_rows failed ({rc})")
    return out


def e2m1_decode(nibbles) -> np.ndarray:
    """E2M1 codes (low 4 bits of each byte) -> float64: +-{0, 0.5, 1, 1.5, 2, 3, 4, 6}."""
    nib = np.ascontiguousarray(nibbles, dtype=np.uint8)
    out = np.empty(nib.shape, dtype=np.float64)
    _load().kx_oracle_e2m1_decode(_ptr(nib), _ptr(out), nib.size)
    return out


def e2m1_encode(x) -> np.ndarray:
    """binary32 -> nearest E2M1 code, ties to the even code, saturating at +-6."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint8)
    _load().kx_oracle_e2m1_encode(_ptr(x), _ptr(out), x.size)
    return out


def quantize_rows_nvfp4(Z, gs: float):
    """4-bit block-scaled code book of BF16 rows (the format of the Section 4.3 task): per 16 consecutive
    elements s = e4m3(max|z| / (6 gs)), q = e2m1(z / (e4m3_value(s) gs)), every step in binary32.
    Z uint16 BF16 bits [rows, cols] -> (Q uint8 [rows, cols / 2] two codes per byte, low nibble first,
    S uint8 [rows, ceil(cols / 16)] E4M3 bytes)."""
    rows, cols = Z.shape
    Z = _bits(Z, (rows, cols), "Z")
    Q = np.empty((rows, cols // 2), dtype=np.uint8)
    S = np.empty((rows, (cols + 15) // 16), dtype=np.uint8)
    rc = _load().kx_oracle_quantize_rows_nvfp4(_ptr(Z), rows, cols, ctypes.c_float(gs), _ptr(Q), _ptr(S))
    if rc != 0:
        raise RuntimeError(f"kx_oracle_quantize_rows_nvfp4 failed ({rc})")
    return Q, S


def outproj_nvfp4(Xq, sx, Wq, sw, alpha: float, bias=None, R=None, rows=None):
    """y = alpha * sum_j e4m3(sx[m,j]) e4m3(sw[n,j]) (Xq[m, block j] . Wq[n, block j]) + bias + R on packed E2M1
    codes with one E4M3 scale per 16 elements; float64, unrounded."""
    M, kb = Xq.shape
    N = Wq.shape[0]
    K = 2 * kb
    nb = (K + 15) // 16
    Xq = _typed(Xq, np.uint8, (M, kb), "Xq")
    Wq = _typed(Wq, np.uint8, (N, kb), "Wq")
    sx = _typed(sx, np.uint8, (M, nb), "sx")
    sw = _typed(sw, np.uint8, (N, nb), "sw")
    bias = _bits(bias, (N,), "bias")
    R = _bits(R, (M, N), "R")
    rows_arr, nrows = _rows_arg(rows, M)
    out = np.empty((nrows, N), dtype=np.float64)
    rc = _load().kx_oracle_outproj_nvfp4_rows(_ptr(Xq), _ptr(sx), _ptr(Wq), _ptr(sw), ctypes.c_double(alpha), _ptr(bias),
                                              _ptr(R), _ptr(rows_arr), nrows, _ptr(out), M, N, K)
    if rc != 0:
        raise RuntimeError(f"kx_oracle_outproj_nvfp4_rows failed ({rc})")
    return out


def swiglu_mx(Xq, ex, Wgq, eg, Wuq, eu, rows=None):
    """z = silu(g) * u with g, u the block-scaled FP8 products of Xq with the gate and the up weights (the
    gate/up step of Appendix A, Algorithm 7, on block-scaled operands); float64, unrounded.  Two calls of
    the block-scaled projection and the activation written out."""
    g = outproj_mx(Xq, ex, Wgq, eg, rows=rows)
    u = outproj_mx(Xq, ex, Wuq, eu, rows=rows)
    return g / (1.0 + np.exp(-g)) * u



def swiglu_nvfp4(Xq, sx, Wgq, sg, Wuq, su, alpha_g: float, alpha_u: float, rows=None):
    """z = silu(g) * u with g = alpha_g * (block-scaled 4-bit product of Xq with the gate weights), u likewise with the
    up weights; float64, unrounded.  Two calls of the 4-bit projection and the activation written out."""
    g = outproj_nvfp4(Xq, sx, Wgq, sg, alpha_g, rows=rows)
    u = outproj_nvfp4(Xq, sx, Wuq, su, alpha_u, rows=rows)
    return g / (1.0 + np.exp(-g)) * u
