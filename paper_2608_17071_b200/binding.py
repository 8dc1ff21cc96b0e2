"""Thin ctypes binding over libkx.so — argument marshalling only.

Every function has the name of the C entry point it calls (see ``include/kx.h``);
all arithmetic runs in the CUDA kernels behind the C ABI.  Tensors may be
``torch`` CUDA tensors of dtype bfloat16 (contiguous) or raw integer device
addresses.  If the shared library is missing this module raises: there is no
fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libkx.so")

KX_OK = 0
KX_ERR_NULL, KX_ERR_SHAPE, KX_ERR_ALIGN, KX_ERR_OVERLAP = 1, 2, 3, 4
KX_ERR_ARCH, KX_ERR_CUDA, KX_ERR_WORKSPACE, KX_ERR_DEVICE_TIMEOUT, KX_ERR_PLAN = 5, 6, 7, 8, 9
KX_ERR_LIMIT = 10
KX_PATH_AUTO, KX_PATH_TILE, KX_PATH_SWAP, KX_PATH_GEMV, KX_PATH_SKINNY = 0, 1, 2, 3, 4

EXPORTS = (
    "kx_init", "kx_shutdown", "kx_outproj_residual", "kx_gemm_bf16", "kx_outproj_residual_ex",
    "kx_outproj_residual_host", "kx_outproj_residual_noalloc", "kx_outproj_residual_strided", "kx_outproj_residual_batched", "kx_rmsnorm", "kx_outproj_residual_rmsnorm",
    "kx_gate_up_swiglu",
    "kx_quantize_rows_int8", "kx_quantize_gate_up_int8", "kx_rmsnorm_quantize_int8", "kx_gate_up_swiglu_int8",
    "kx_outproj_residual_int8",
    "kx_quantize_rows_fp8", "kx_quantize_gate_up_fp8", "kx_rmsnorm_quantize_fp8", "kx_gate_up_swiglu_fp8",
    "kx_outproj_residual_fp8",
    "kx_mx_scale_bytes", "kx_quantize_rows_mxfp8", "kx_rmsnorm_quantize_mxfp8", "kx_outproj_residual_mxfp8", "kx_outproj_residual_mxfp8_ex",
    "kx_quantize_gate_up_mxfp8", "kx_gate_up_swiglu_mxfp8",
    "kx_nvfp4_scale_bytes", "kx_quantize_rows_nvfp4", "kx_outproj_residual_nvfp4",
    "kx_rmsnorm_quantize_nvfp4", "kx_quantize_gate_up_nvfp4", "kx_gate_up_swiglu_nvfp4",
    "kx_plan_query", "kx_last_device_status", "kx_status_string",
    "kx_version",
)


class PlanOverride(ctypes.Structure):
    _fields_ = [
        ("path", ctypes.c_int32), ("block_n", ctypes.c_int32), ("cta_pair", ctypes.c_int32),
        ("split_k", ctypes.c_int32), ("raster_group", ctypes.c_int32), ("max_ctas", ctypes.c_int32),
        ("spin_limit_us", ctypes.c_int32), ("debug_drop_kblocks", ctypes.c_int32),
        ("stages", ctypes.c_int32), ("stream_k", ctypes.c_int32), ("narrow_tail", ctypes.c_int32), ("no_pdl", ctypes.c_int32), ("cluster_reduce", ctypes.c_int32), ("no_table", ctypes.c_int32), ("k_cluster", ctypes.c_int32), ("l2_prefetch", ctypes.c_int32),
    ]


class PlanInfo(ctypes.Structure):
    _fields_ = [
        ("path", ctypes.c_int32), ("block_n", ctypes.c_int32), ("cta_pair", ctypes.c_int32),
        ("stages", ctypes.c_int32), ("split_k", ctypes.c_int32), ("raster_group", ctypes.c_int32),
        ("grid", ctypes.c_int32), ("tiles", ctypes.c_int32), ("launches", ctypes.c_int32),
        ("smem_bytes", ctypes.c_int32), ("workspace_bytes", ctypes.c_int64),
        ("stream_k", ctypes.c_int32), ("narrow_tiles", ctypes.c_int32), ("cluster_reduce", ctypes.c_int32), ("from_table", ctypes.c_int32),
    ]


class KxError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {kx_status_string(status)}")


_lib = None


def load():
    """Load libkx.so.  Raises if it has not been built: no fallback exists."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_17071_b200.build` "
            "(the CUDA library is the only implementation; there is no fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
    lib.kx_init.argtypes = [ci]
    lib.kx_shutdown.argtypes = []
    lib.kx_outproj_residual.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp]
    lib.kx_gemm_bf16.argtypes = [vp, vp, vp, i64, i64, i64, vp]
    lib.kx_outproj_residual_ex.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp, ctypes.POINTER(PlanOverride)]
    lib.kx_outproj_residual_host.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp]
    lib.kx_outproj_residual_noalloc.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp]
    lib.kx_outproj_residual_strided.argtypes = [vp, i64, vp, i64, vp, vp, i64, vp, i64, i64, i64, i64, vp]
    lib.kx_outproj_residual_batched.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, i64, i64, i64, i64, vp]
    lib.kx_rmsnorm.argtypes = [vp, vp, ctypes.c_float, vp, i64, i64, vp]
    lib.kx_gate_up_swiglu.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp]
    lib.kx_outproj_residual_rmsnorm.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, i64, i64, i64, vp]
    lib.kx_quantize_rows_int8.argtypes = [vp, vp, vp, i64, i64, vp]
    lib.kx_quantize_gate_up_int8.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, vp]
    lib.kx_rmsnorm_quantize_int8.argtypes = [vp, vp, ctypes.c_float, vp, vp, i64, i64, vp]
    lib.kx_gate_up_swiglu_int8.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp]
    lib.kx_outproj_residual_int8.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp]
    for sfx in ("fp8",):
        getattr(lib, f"kx_quantize_rows_{sfx}").argtypes = lib.kx_quantize_rows_int8.argtypes
        getattr(lib, f"kx_quantize_gate_up_{sfx}").argtypes = lib.kx_quantize_gate_up_int8.argtypes
        getattr(lib, f"kx_rmsnorm_quantize_{sfx}").argtypes = lib.kx_rmsnorm_quantize_int8.argtypes
        getattr(lib, f"kx_gate_up_swiglu_{sfx}").argtypes = lib.kx_gate_up_swiglu_int8.argtypes
        getattr(lib, f"kx_outproj_residual_{sfx}").argtypes = lib.kx_outproj_residual_int8.argtypes
    lib.kx_mx_scale_bytes.argtypes = [i64, i64]
    lib.kx_quantize_rows_mxfp8.argtypes = [vp, vp, vp, i64, i64, vp]
    lib.kx_rmsnorm_quantize_mxfp8.argtypes = [vp, vp, ctypes.c_float, vp, vp, i64, i64, vp]
    lib.kx_outproj_residual_mxfp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp]
    lib.kx_outproj_residual_mxfp8_ex.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, ctypes.POINTER(PlanOverride)]
    lib.kx_quantize_gate_up_mxfp8.argtypes = [vp, vp, vp, vp, vp, i64, i64, vp]
    lib.kx_gate_up_swiglu_mxfp8.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, vp]
    lib.kx_nvfp4_scale_bytes.argtypes = [i64, i64]
    lib.kx_quantize_rows_nvfp4.argtypes = [vp, ctypes.c_float, vp, vp, i64, i64, vp]
    lib.kx_outproj_residual_nvfp4.argtypes = [vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, i64, i64, i64, vp,
                                              ctypes.POINTER(PlanOverride)]
    cf = ctypes.c_float
    lib.kx_rmsnorm_quantize_nvfp4.argtypes = [vp, vp, cf, cf, vp, vp, i64, i64, vp]
    lib.kx_quantize_gate_up_nvfp4.argtypes = [vp, vp, cf, cf, vp, vp, vp, i64, i64, vp]
    lib.kx_gate_up_swiglu_nvfp4.argtypes = [vp, vp, vp, vp, vp, cf, cf, vp, i64, i64, i64, vp]
    lib.kx_plan_query.argtypes = [i64, i64, i64, ci, ci, ctypes.POINTER(PlanOverride), ctypes.POINTER(PlanInfo)]
    lib.kx_last_device_status.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.kx_status_string.argtypes = [ci]
    lib.kx_status_string.restype = ctypes.c_char_p
    lib.kx_version.argtypes = []
    for name in EXPORTS:
        if name in ("kx_mx_scale_bytes", "kx_nvfp4_scale_bytes"):
            getattr(lib, name).restype = i64
        elif name != "kx_status_string":
            getattr(lib, name).restype = ci
    _lib = lib
    return lib


def _addr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return int(t.data_ptr())


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream) or None
    if isinstance(stream, int):
        return stream or None
    return int(stream.cuda_stream) or None


def _check_bf16(name, t, shape):
    import torch
    if t is None or isinstance(t, int):
        return
    if t.dtype != torch.bfloat16 or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: need a contiguous bfloat16 tensor of shape {tuple(shape)}, "
                         f"got {t.dtype} {tuple(t.shape)} contiguous={t.is_contiguous()}")


def _check(name, t, shape, dtype):
    if t is None or isinstance(t, int):
        return
    if t.dtype != dtype or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: need a contiguous {dtype} tensor of shape {tuple(shape)}, "
                         f"got {t.dtype} {tuple(t.shape)} contiguous={t.is_contiguous()}")


def make_override(**kw) -> PlanOverride:
    ov = PlanOverride()
    for k, v in kw.items():
        if not hasattr(ov, k):
            raise TypeError(f"unknown plan override field {k!r}")
        setattr(ov, k, int(v))
    return ov


def kx_version() -> int:
    return int(load().kx_version())


def kx_status_string(status: int) -> str:
    return load().kx_status_string(int(status)).decode()


def kx_init(device: int = 0) -> None:
    rc = load().kx_init(int(device))
    if rc != KX_OK:
        raise KxError(rc, "kx_init")


def kx_shutdown() -> None:
    load().kx_shutdown()


def kx_outproj_residual(X, W, bias, R, Y, stream=None, M=None, N=None, K=None, check=True) -> int:
    """Y = X W^T (+ bias) + R on the current stream.  Shapes come from the tensors
    unless M, N, K are given (raw-pointer use)."""
    if M is None:
        M, K = X.shape
        N = W.shape[0]
        _check_bf16("X", X, (M, K)); _check_bf16("W", W, (N, K)); _check_bf16("bias", bias, (N,))
        _check_bf16("R", R, (M, N)); _check_bf16("Y", Y, (M, N))
    rc = load().kx_outproj_residual(_addr(X), _addr(W), _addr(bias), _addr(R), _addr(Y), M, N, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual")
    return rc


def kx_gemm_bf16(X, W, Y, stream=None, M=None, N=None, K=None, check=True) -> int:
    """Y = X W^T on the current stream."""
    if M is None:
        M, K = X.shape
        N = W.shape[0]
        _check_bf16("X", X, (M, K)); _check_bf16("W", W, (N, K)); _check_bf16("Y", Y, (M, N))
    rc = load().kx_gemm_bf16(_addr(X), _addr(W), _addr(Y), M, N, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_gemm_bf16")
    return rc


def kx_outproj_residual_ex(X, W, bias, R, Y, ov: Optional[PlanOverride] = None, stream=None,
                           M=None, N=None, K=None, check=True) -> int:
    """As kx_outproj_residual (bias and R optional) with an explicit plan override."""
    if M is None:
        M, K = X.shape
        N = W.shape[0]
        _check_bf16("X", X, (M, K)); _check_bf16("W", W, (N, K)); _check_bf16("bias", bias, (N,))
        _check_bf16("R", R, (M, N)); _check_bf16("Y", Y, (M, N))
    rc = load().kx_outproj_residual_ex(_addr(X), _addr(W), _addr(bias), _addr(R), _addr(Y), M, N, K,
                                       _stream(stream), ctypes.byref(ov) if ov is not None else None)
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual_ex")
    return rc


def kx_outproj_residual_noalloc(X, W, bias, R, Y, stream=None, M=None, N=None, K=None, check=True) -> int:
    """Small-M form that never allocates: for callers that may not ask the driver
    for device memory (a process whose framework owns all of HBM, a loop that cannot
    afford an allocation's synchronisation).  Its scratch is a fixed array inside the
    library; M <= 256, N <= 524288, otherwise KX_ERR_LIMIT.  bias and R may be None.
    Calls that overlap on the GPU share that array and would race."""
    if M is None:
        M, K = X.shape
        N = W.shape[0]
        _check_bf16("X", X, (M, K)); _check_bf16("W", W, (N, K)); _check_bf16("bias", bias, (N,))
        _check_bf16("R", R, (M, N)); _check_bf16("Y", Y, (M, N))
    rc = load().kx_outproj_residual_noalloc(_addr(X), _addr(W), _addr(bias), _addr(R), _addr(Y), M, N, K,
                                            _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual_noalloc")
    return rc


def kx_gate_up_swiglu(X, Wg, Wu, Z, stream=None, M=None, I=None, K=None, check=True) -> int:
    """Z = silu(X Wg^T) * (X Wu^T) with the SwiGLU product fused into the GEMM epilogue."""
    if M is None:
        M, K = X.shape
        I = Wg.shape[0]
        _check_bf16("X", X, (M, K)); _check_bf16("Wg", Wg, (I, K)); _check_bf16("Wu", Wu, (I, K))
        _check_bf16("Z", Z, (M, I))
    rc = load().kx_gate_up_swiglu(_addr(X), _addr(Wg), _addr(Wu), _addr(Z), M, I, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_gate_up_swiglu")
    return rc


def _code_dtype(fmt):
    import torch
    if fmt == "int8":
        return torch.int8
    if fmt == "fp8":
        return torch.float8_e4m3fn
    raise ValueError(f"unknown 8-bit format {fmt!r} (int8 or fp8)")


def _check_rows(name, t, shape):
    import torch
    if t is None:
        return 0
    if t.dtype != torch.bfloat16 or tuple(t.shape) != tuple(shape) or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name}: need a bfloat16 tensor of shape {tuple(shape)} with unit column stride, "
                         f"got {t.dtype} {tuple(t.shape)} strides {tuple(t.stride())}")
    return int(t.stride(0))


def kx_outproj_residual_strided(X, W, bias, R, Y, stream=None, check=True) -> int:
    """kx_outproj_residual on row-pitched views (column stride 1, any row stride that is a multiple of 8)."""
    M, K = X.shape
    N = W.shape[0]
    ldx, ldw = _check_rows("X", X, (M, K)), _check_rows("W", W, (N, K))
    ldr, ldy = _check_rows("R", R, (M, N)), _check_rows("Y", Y, (M, N))
    _check_bf16("bias", bias, (N,))
    rc = load().kx_outproj_residual_strided(_addr(X), ldx, _addr(W), ldw, _addr(bias), _addr(R), ldr, _addr(Y), ldy,
                                            M, N, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual_strided")
    return rc


def kx_outproj_residual_batched(X, W, bias, R, Y, stream=None, check=True) -> int:
    """`batch` problems: X [B,M,K], W [B,N,K] or [N,K] (shared), bias [B,N] / [N] / None, R [B,M,N] / None,
    Y [B,M,N]; contiguous bfloat16 tensors."""
    B, M, K = X.shape
    shared_w = W.dim() == 2
    N = W.shape[-2]
    _check_bf16("X", X, (B, M, K)); _check_bf16("W", W, (N, K) if shared_w else (B, N, K))
    _check_bf16("R", R, (B, M, N)); _check_bf16("Y", Y, (B, M, N))
    sb = 0
    if bias is not None:
        shared_b = bias.dim() == 1
        _check_bf16("bias", bias, (N,) if shared_b else (B, N))
        sb = 0 if shared_b else N
    rc = load().kx_outproj_residual_batched(_addr(X), M * K, _addr(W), 0 if shared_w else N * K, _addr(bias), sb,
                                            _addr(R), M * N, _addr(Y), M * N, M, N, K, B, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual_batched")
    return rc


def kx_quantize_rows_int8(A, Q, S, stream=None, check=True, fmt="int8") -> int:
    """Q (int8), S (float32 per row) = symmetric per-row INT8 code book of the BF16 matrix A."""
    import torch
    rows, cols = A.shape
    _check_bf16("A", A, (rows, cols)); _check("Q", Q, (rows, cols), _code_dtype(fmt)); _check("S", S, (rows,), torch.float32)
    rc = getattr(load(), f"kx_quantize_rows_{fmt}")(_addr(A), _addr(Q), _addr(S), rows, cols, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, f"kx_quantize_rows_{fmt}")
    return rc


def kx_quantize_gate_up_int8(Wg, Wu, Qg, Sg, Qu, Su, stream=None, check=True, fmt="int8") -> int:
    """Code books of the gate and the up weight matrices in one launch."""
    import torch
    I, K = Wg.shape
    _check_bf16("Wg", Wg, (I, K)); _check_bf16("Wu", Wu, (I, K))
    _check("Qg", Qg, (I, K), _code_dtype(fmt)); _check("Qu", Qu, (I, K), _code_dtype(fmt))
    _check("Sg", Sg, (I,), torch.float32); _check("Su", Su, (I,), torch.float32)
    rc = getattr(load(), f"kx_quantize_gate_up_{fmt}")(_addr(Wg), _addr(Wu), _addr(Qg), _addr(Sg), _addr(Qu), _addr(Su),
                                                       I, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, f"kx_quantize_gate_up_{fmt}")
    return rc


def kx_rmsnorm_quantize_int8(H, gamma, eps: float, Q, S, stream=None, check=True, fmt="int8") -> int:
    """Q, S = code book of RMSNorm(H) * gamma (rounded to BF16 as kx_rmsnorm would), H read once."""
    import torch
    M, N = H.shape
    _check_bf16("H", H, (M, N)); _check_bf16("gamma", gamma, (N,))
    _check("Q", Q, (M, N), _code_dtype(fmt)); _check("S", S, (M,), torch.float32)
    rc = getattr(load(), f"kx_rmsnorm_quantize_{fmt}")(_addr(H), _addr(gamma), float(eps), _addr(Q), _addr(S), M, N,
                                                       _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, f"kx_rmsnorm_quantize_{fmt}")
    return rc


def kx_gate_up_swiglu_int8(Xq, sx, Wgq, sg, Wuq, su, Z, stream=None, check=True, fmt="int8") -> int:
    """Z = silu((Xq Wgq^T) sx sg) * ((Xq Wuq^T) sx su): INT8 GEMM, dequantisation and SwiGLU fused."""
    import torch
    M, K = Xq.shape
    I = Wgq.shape[0]
    cd = _code_dtype(fmt)
    _check("Xq", Xq, (M, K), cd); _check("Wgq", Wgq, (I, K), cd); _check("Wuq", Wuq, (I, K), cd)
    _check("sx", sx, (M,), torch.float32); _check("sg", sg, (I,), torch.float32); _check("su", su, (I,), torch.float32)
    _check_bf16("Z", Z, (M, I))
    rc = getattr(load(), f"kx_gate_up_swiglu_{fmt}")(_addr(Xq), _addr(sx), _addr(Wgq), _addr(sg), _addr(Wuq), _addr(su),
                                                     _addr(Z), M, I, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, f"kx_gate_up_swiglu_{fmt}")
    return rc


def kx_outproj_residual_int8(Xq, sx, Wq, sw, bias, R, Y, stream=None, check=True, fmt="int8") -> int:
    """Y = (Xq Wq^T) sx sw + bias + R on INT8 codes; bias / R may be None; R may be Y."""
    import torch
    M, K = Xq.shape
    N = Wq.shape[0]
    _check("Xq", Xq, (M, K), _code_dtype(fmt)); _check("Wq", Wq, (N, K), _code_dtype(fmt))
    _check("sx", sx, (M,), torch.float32); _check("sw", sw, (N,), torch.float32)
    _check_bf16("bias", bias, (N,)); _check_bf16("R", R, (M, N)); _check_bf16("Y", Y, (M, N))
    rc = getattr(load(), f"kx_outproj_residual_{fmt}")(_addr(Xq), _addr(sx), _addr(Wq), _addr(sw), _addr(bias), _addr(R),
                                                       _addr(Y), M, N, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, f"kx_outproj_residual_{fmt}")
    return rc


def kx_quantize_rows_fp8(A, Q, S, **kw) -> int:
    """FP8 E4M3 twin of kx_quantize_rows_int8 (Q is a float8_e4m3fn tensor)."""
    return kx_quantize_rows_int8(A, Q, S, fmt="fp8", **kw)


def kx_quantize_gate_up_fp8(Wg, Wu, Qg, Sg, Qu, Su, **kw) -> int:
    return kx_quantize_gate_up_int8(Wg, Wu, Qg, Sg, Qu, Su, fmt="fp8", **kw)


def kx_rmsnorm_quantize_fp8(H, gamma, eps: float, Q, S, **kw) -> int:
    return kx_rmsnorm_quantize_int8(H, gamma, eps, Q, S, fmt="fp8", **kw)


def kx_gate_up_swiglu_fp8(Xq, sx, Wgq, sg, Wuq, su, Z, **kw) -> int:
    return kx_gate_up_swiglu_int8(Xq, sx, Wgq, sg, Wuq, su, Z, fmt="fp8", **kw)


def kx_outproj_residual_fp8(Xq, sx, Wq, sw, bias, R, Y, **kw) -> int:
    return kx_outproj_residual_int8(Xq, sx, Wq, sw, bias, R, Y, fmt="fp8", **kw)


def kx_rmsnorm(H, gamma, eps: float, Z, stream=None, M=None, N=None, check=True) -> int:
    """Z = RMSNorm(H) * gamma over the rows of H (BF16, FP32 arithmetic); Z may be H."""
    if M is None:
        M, N = H.shape
        _check_bf16("H", H, (M, N)); _check_bf16("gamma", gamma, (N,)); _check_bf16("Z", Z, (M, N))
    rc = load().kx_rmsnorm(_addr(H), _addr(gamma), float(eps), _addr(Z), M, N, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_rmsnorm")
    return rc


def kx_outproj_residual_rmsnorm(X, W, bias, R, gamma, eps: float, H, Z, stream=None, M=None, N=None, K=None,
                                check=True) -> int:
    """H = X W^T (+ bias) + R and Z = RMSNorm(H) * gamma, two kernels on one stream."""
    if M is None:
        M, K = X.shape
        N = W.shape[0]
        _check_bf16("X", X, (M, K)); _check_bf16("W", W, (N, K)); _check_bf16("bias", bias, (N,))
        _check_bf16("R", R, (M, N)); _check_bf16("gamma", gamma, (N,))
        _check_bf16("H", H, (M, N)); _check_bf16("Z", Z, (M, N))
    rc = load().kx_outproj_residual_rmsnorm(_addr(X), _addr(W), _addr(bias), _addr(R), _addr(gamma), float(eps),
                                            _addr(H), _addr(Z), M, N, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual_rmsnorm")
    return rc


def bound_call(X, W, bias, R, Y, stream=None, plain: bool = False, ov: Optional[PlanOverride] = None):
    """Marshal the arguments of kx_outproj_residual (or kx_gemm_bf16 when `plain`)
    once and return a zero-argument callable that enqueues that same C call.
    For callers that repeat one call many times (the Python-side checks and pointer
    extraction cost more than a small kernel runs).  The callable holds references to
    the tensors, so their memory stays allocated for as long as it is alive."""
    M, K = X.shape
    N = W.shape[0]
    _check_bf16("X", X, (M, K)); _check_bf16("W", W, (N, K)); _check_bf16("Y", Y, (M, N))
    lib = load()
    vp = ctypes.c_void_p
    st = vp(_stream(stream))
    if ov is not None:
        # explicit plan: kx_outproj_residual_ex (bias and R optional)
        _check_bf16("bias", bias, (N,)); _check_bf16("R", R, (M, N))
        args = (vp(_addr(X)), vp(_addr(W)), vp(_addr(bias)), vp(_addr(R)), vp(_addr(Y)),
                ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_int64(K), st, ctypes.byref(ov))
        fn = lib.kx_outproj_residual_ex
    elif plain:
        args = (vp(_addr(X)), vp(_addr(W)), vp(_addr(Y)), ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_int64(K), st)
        fn = lib.kx_gemm_bf16
    else:
        _check_bf16("bias", bias, (N,)); _check_bf16("R", R, (M, N))
        args = (vp(_addr(X)), vp(_addr(W)), vp(_addr(bias)), vp(_addr(R)), vp(_addr(Y)),
                ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_int64(K), st)
        fn = lib.kx_outproj_residual

    keep = (X, W, bias, R, Y, stream, ov)

    def run(_keep=keep):
        rc = fn(*args)
        if rc != KX_OK:
            raise KxError(rc, fn.__name__)
    run.tensors = keep
    # the same call bound to another stream (a capture stream, for instance)
    run.rebind = lambda new_stream: bound_call(X, W, bias, R, Y, stream=new_stream, plain=plain, ov=ov)
    return run


def kx_outproj_residual_host(X, W, bias, R, Y, M: int, N: int, K: int, stream=None, check=True) -> int:
    """Host-buffer form: X, W, bias, R, Y are HOST addresses (ints) or CPU tensors /
    numpy arrays holding BF16 bits; copies in, runs, copies Y back, synchronises."""
    def host_addr(a):
        if a is None or isinstance(a, int):
            return a
        if hasattr(a, "data_ptr"):
            return int(a.data_ptr())
        return int(a.ctypes.data)
    rc = load().kx_outproj_residual_host(host_addr(X), host_addr(W), host_addr(bias), host_addr(R),
                                         host_addr(Y), M, N, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual_host")
    return rc


def kx_plan_query(M: int, N: int, K: int, has_bias: bool = True, has_residual: bool = True,
                  ov: Optional[PlanOverride] = None) -> PlanInfo:
    info = PlanInfo()
    rc = load().kx_plan_query(M, N, K, int(has_bias), int(has_residual),
                              ctypes.byref(ov) if ov is not None else None, ctypes.byref(info))
    if rc != KX_OK:
        raise KxError(rc, "kx_plan_query")
    return info


def kx_last_device_status(stream=None):
    """(code, detail) after synchronising the stream; clears the status word."""
    code, detail = ctypes.c_int(0), ctypes.c_int(0)
    rc = load().kx_last_device_status(_stream(stream), ctypes.byref(code), ctypes.byref(detail))
    if rc != KX_OK:
        raise KxError(rc, "kx_last_device_status")
    return code.value, detail.value


def kx_mx_scale_bytes(rows: int, cols: int) -> int:
    """Bytes of the chunked E8M0 scale array of a [rows, cols] block-scaled matrix."""
    return int(load().kx_mx_scale_bytes(int(rows), int(cols)))


def kx_quantize_rows_mxfp8(A, Q, SF, stream=None, check=True) -> int:
    """Q (float8_e4m3fn [rows, cols]), SF (uint8, kx_mx_scale_bytes(rows, cols) bytes, chunked layout) =
    block-scaled FP8 code book of the BF16 matrix A (one E8M0 scale per 32 elements of a row)."""
    import torch
    rows, cols = A.shape
    _check_bf16("A", A, (rows, cols)); _check("Q", Q, (rows, cols), torch.float8_e4m3fn)
    _check("SF", SF, (kx_mx_scale_bytes(rows, cols),), torch.uint8)
    rc = load().kx_quantize_rows_mxfp8(_addr(A), _addr(Q), _addr(SF), rows, cols, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_quantize_rows_mxfp8")
    return rc


def kx_rmsnorm_quantize_mxfp8(H, gamma, eps: float, Q, SF, stream=None, check=True) -> int:
    """Q, SF = block-scaled FP8 code book of RMSNorm(H) * gamma (rounded to BF16 as kx_rmsnorm would), H read once."""
    import torch
    M, N = H.shape
    _check_bf16("H", H, (M, N)); _check_bf16("gamma", gamma, (N,)); _check("Q", Q, (M, N), torch.float8_e4m3fn)
    _check("SF", SF, (kx_mx_scale_bytes(M, N),), torch.uint8)
    rc = load().kx_rmsnorm_quantize_mxfp8(_addr(H), _addr(gamma), float(eps), _addr(Q), _addr(SF), M, N, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_rmsnorm_quantize_mxfp8")
    return rc


def kx_outproj_residual_mxfp8(Xq, SFX, Wq, SFW, bias, R, Y, stream=None, check=True, override=None) -> int:
    """Y = block-scaled (Xq, SFX) (Wq, SFW)^T + bias + R; bias / R may be None; R may be Y.
    override: a PlanOverride (block_n, cta_pair, raster_group) or None."""
    import torch
    M, K = Xq.shape
    N = Wq.shape[0]
    _check("Xq", Xq, (M, K), torch.float8_e4m3fn); _check("Wq", Wq, (N, K), torch.float8_e4m3fn)
    _check("SFX", SFX, (kx_mx_scale_bytes(M, K),), torch.uint8); _check("SFW", SFW, (kx_mx_scale_bytes(N, K),), torch.uint8)
    _check_bf16("bias", bias, (N,)); _check_bf16("R", R, (M, N)); _check_bf16("Y", Y, (M, N))
    if override is None:
        rc = load().kx_outproj_residual_mxfp8(_addr(Xq), _addr(SFX), _addr(Wq), _addr(SFW), _addr(bias), _addr(R), _addr(Y),
                                              M, N, K, _stream(stream))
    else:
        rc = load().kx_outproj_residual_mxfp8_ex(_addr(Xq), _addr(SFX), _addr(Wq), _addr(SFW), _addr(bias), _addr(R),
                                                 _addr(Y), M, N, K, _stream(stream), ctypes.byref(override))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual_mxfp8")
    return rc


def kx_quantize_gate_up_mxfp8(Wg, Wu, Qg, Qu, SFGU, stream=None, check=True) -> int:
    """Block-scaled code books of the gate and the up weights; SFGU = gate scales followed by up scales."""
    import torch
    I, K = Wg.shape
    _check_bf16("Wg", Wg, (I, K)); _check_bf16("Wu", Wu, (I, K))
    _check("Qg", Qg, (I, K), torch.float8_e4m3fn); _check("Qu", Qu, (I, K), torch.float8_e4m3fn)
    _check("SFGU", SFGU, (2 * kx_mx_scale_bytes(I, K),), torch.uint8)
    rc = load().kx_quantize_gate_up_mxfp8(_addr(Wg), _addr(Wu), _addr(Qg), _addr(Qu), _addr(SFGU), I, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_quantize_gate_up_mxfp8")
    return rc


def kx_gate_up_swiglu_mxfp8(Xq, SFX, Wgq, Wuq, SFGU, Z, stream=None, check=True) -> int:
    """Z = silu(g) * u on block-scaled FP8 operands (g / u = products of Xq with the gate / up weights)."""
    import torch
    M, K = Xq.shape
    I = Wgq.shape[0]
    _check("Xq", Xq, (M, K), torch.float8_e4m3fn); _check("Wgq", Wgq, (I, K), torch.float8_e4m3fn)
    _check("Wuq", Wuq, (I, K), torch.float8_e4m3fn); _check("SFX", SFX, (kx_mx_scale_bytes(M, K),), torch.uint8)
    _check("SFGU", SFGU, (2 * kx_mx_scale_bytes(I, K),), torch.uint8); _check_bf16("Z", Z, (M, I))
    rc = load().kx_gate_up_swiglu_mxfp8(_addr(Xq), _addr(SFX), _addr(Wgq), _addr(Wuq), _addr(SFGU), _addr(Z), M, I, K,
                                        _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_gate_up_swiglu_mxfp8")
    return rc


def kx_nvfp4_scale_bytes(rows: int, cols: int) -> int:
    """Bytes of the chunked E4M3 scale array of a [rows, cols] 4-bit block-scaled matrix."""
    return int(load().kx_nvfp4_scale_bytes(int(rows), int(cols)))


def kx_quantize_rows_nvfp4(A, gs: float, Q, SF, stream=None, check=True) -> int:
    """Q (uint8 [rows, cols / 2], two E2M1 codes per byte), SF (uint8, kx_nvfp4_scale_bytes(rows, cols) bytes) =
    4-bit block-scaled code book of the BF16 matrix A with tensor scale gs."""
    import torch
    rows, cols = A.shape
    _check_bf16("A", A, (rows, cols)); _check("Q", Q, (rows, cols // 2), torch.uint8)
    _check("SF", SF, (kx_nvfp4_scale_bytes(rows, cols),), torch.uint8)
    rc = load().kx_quantize_rows_nvfp4(_addr(A), float(gs), _addr(Q), _addr(SF), rows, cols, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_quantize_rows_nvfp4")
    return rc


def kx_outproj_residual_nvfp4(Xq, SFX, Wq, SFW, alpha: float, bias, R, Y, stream=None, check=True, override=None) -> int:
    """Y = alpha * block-scaled (Xq, SFX) (Wq, SFW)^T + bias + R on packed E2M1 codes; bias / R may be None."""
    import torch
    M, kb = Xq.shape
    N = Wq.shape[0]
    K = 2 * kb
    _check("Xq", Xq, (M, kb), torch.uint8); _check("Wq", Wq, (N, kb), torch.uint8)
    _check("SFX", SFX, (kx_nvfp4_scale_bytes(M, K),), torch.uint8); _check("SFW", SFW, (kx_nvfp4_scale_bytes(N, K),), torch.uint8)
    _check_bf16("bias", bias, (N,)); _check_bf16("R", R, (M, N)); _check_bf16("Y", Y, (M, N))
    rc = load().kx_outproj_residual_nvfp4(_addr(Xq), _addr(SFX), _addr(Wq), _addr(SFW), float(alpha), _addr(bias), _addr(R),
                                          _addr(Y), M, N, K, _stream(stream),
                                          ctypes.byref(override) if override is not None else None)
    if check and rc != KX_OK:
        raise KxError(rc, "kx_outproj_residual_nvfp4")
    return rc


def kx_rmsnorm_quantize_nvfp4(H, gamma, eps: float, gs: float, Q, SF, stream=None, check=True) -> int:
    """Q, SF = 4-bit block-scaled code book of RMSNorm(H) * gamma (rounded to BF16 as kx_rmsnorm would) with tensor scale gs."""
    import torch
    M, N = H.shape
    _check_bf16("H", H, (M, N)); _check_bf16("gamma", gamma, (N,)); _check("Q", Q, (M, N // 2), torch.uint8)
    _check("SF", SF, (kx_nvfp4_scale_bytes(M, N),), torch.uint8)
    rc = load().kx_rmsnorm_quantize_nvfp4(_addr(H), _addr(gamma), float(eps), float(gs), _addr(Q), _addr(SF), M, N,
                                          _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_rmsnorm_quantize_nvfp4")
    return rc


def kx_quantize_gate_up_nvfp4(Wg, Wu, gsg: float, gsu: float, Qg, Qu, SFGU, stream=None, check=True) -> int:
    """4-bit code books of the gate and the up weights; SFGU = gate scales followed by up scales."""
    import torch
    I, K = Wg.shape
    _check_bf16("Wg", Wg, (I, K)); _check_bf16("Wu", Wu, (I, K))
    _check("Qg", Qg, (I, K // 2), torch.uint8); _check("Qu", Qu, (I, K // 2), torch.uint8)
    _check("SFGU", SFGU, (2 * kx_nvfp4_scale_bytes(I, K),), torch.uint8)
    rc = load().kx_quantize_gate_up_nvfp4(_addr(Wg), _addr(Wu), float(gsg), float(gsu), _addr(Qg), _addr(Qu), _addr(SFGU),
                                          I, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_quantize_gate_up_nvfp4")
    return rc


def kx_gate_up_swiglu_nvfp4(Xq, SFX, Wgq, Wuq, SFGU, alpha_g: float, alpha_u: float, Z, stream=None, check=True) -> int:
    """Z = silu(alpha_g g) * (alpha_u u) on packed 4-bit block-scaled operands."""
    import torch
    M, kb = Xq.shape
    I, K = Wgq.shape[0], 2 * kb
    _check("Xq", Xq, (M, kb), torch.uint8); _check("Wgq", Wgq, (I, kb), torch.uint8); _check("Wuq", Wuq, (I, kb), torch.uint8)
    _check("SFX", SFX, (kx_nvfp4_scale_bytes(M, K),), torch.uint8)
    _check("SFGU", SFGU, (2 * kx_nvfp4_scale_bytes(I, K),), torch.uint8); _check_bf16("Z", Z, (M, I))
    rc = load().kx_gate_up_swiglu_nvfp4(_addr(Xq), _addr(SFX), _addr(Wgq), _addr(Wuq), _addr(SFGU), float(alpha_g),
                                        float(alpha_u), _addr(Z), M, I, K, _stream(stream))
    if check and rc != KX_OK:
        raise KxError(rc, "kx_gate_up_swiglu_nvfp4")
    return rc
