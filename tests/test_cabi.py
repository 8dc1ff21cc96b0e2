"""The C-ABI library without a GPU: it builds, loads, exports every symbol the
header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2608_17071_b200 import binding as kx
from paper_2608_17071_b200 import build as kxbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    kxbuild.build()
    return kx.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "kx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kx_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert "kx_outproj_residual" in names and "kx_gemm_bf16" in names and len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/kx.h but not exported"
    assert set(names) == set(kx.EXPORTS)


def test_version_and_status_strings(lib):
    assert kx.kx_version() == 100
    for code in range(0, 11):
        s = kx.kx_status_string(code)
        assert s.startswith("KX_") and "UNKNOWN" not in s
    assert "UNKNOWN" in kx.kx_status_string(99)


def test_struct_layouts_match_header():
    assert ctypes.sizeof(kx.PlanOverride) == 16 * 4
    assert ctypes.sizeof(kx.PlanInfo) == 10 * 4 + 8 + 4 * 4


def test_argument_validation_needs_no_device(lib):
    A = 0x10000  # fake, 16-byte aligned, never dereferenced: validation fails first
    f = lib.kx_outproj_residual
    g = lib.kx_gemm_bf16
    MB = 1 << 20
    X, W, B, R, Y = A, A + 64 * MB, A + 128 * MB, A + 192 * MB, A + 256 * MB
    assert f(X, W, B, R, Y, -1, 8, 8, None) == kx.KX_ERR_SHAPE
    assert f(X, W, B, R, Y, 4, 12, 8, None) == kx.KX_ERR_SHAPE        # N % 8
    assert f(X, W, B, R, Y, 4, 8, 20, None) == kx.KX_ERR_SHAPE        # K % 8
    assert f(X, W, B, R, Y, 1 << 31, 8, 8, None) == kx.KX_ERR_SHAPE
    assert f(X, W, B, R, None, 4, 8, 8, None) == kx.KX_ERR_NULL
    assert f(None, W, B, R, Y, 4, 8, 8, None) == kx.KX_ERR_NULL
    assert f(X, None, B, R, Y, 4, 8, 8, None) == kx.KX_ERR_NULL
    assert f(X, W, B, None, Y, 4, 8, 8, None) == kx.KX_ERR_NULL       # residual is required here
    assert f(X + 2, W, B, R, Y, 4, 8, 8, None) == kx.KX_ERR_ALIGN
    assert f(X, W, B + 8, R, Y, 4, 8, 8, None) == kx.KX_ERR_ALIGN
    assert f(X, W, B, R, Y + 4, 4, 8, 8, None) == kx.KX_ERR_ALIGN
    assert f(X, W, B, R, X, 4, 8, 8, None) == kx.KX_ERR_OVERLAP       # Y aliases X
    assert f(X, W, B, R, W + 16, 4, 8, 8, None) == kx.KX_ERR_OVERLAP  # Y inside W
    assert f(X, W, B, R, R + 16, 4, 8, 8, None) == kx.KX_ERR_OVERLAP  # partial overlap with R
    assert f(X, W, Y, R, Y, 4, 8, 8, None) == kx.KX_ERR_OVERLAP       # Y aliases bias
    # empty problems are successful no-ops and need no pointers
    assert f(None, None, None, None, None, 0, 8, 8, None) == kx.KX_OK
    assert g(None, None, None, 4, 0, 8, None) == kx.KX_OK
    assert g(X, W, Y, 4, 8, 8 + 4, None) == kx.KX_ERR_SHAPE
    assert lib.kx_plan_query(4, 8, 8, 1, 1, None, None) == kx.KX_ERR_NULL
    assert lib.kx_last_device_status(None, None, None) == kx.KX_ERR_NULL
    assert lib.kx_outproj_residual_host(X, W, None, None, None, 4, 8, 8, None) == kx.KX_ERR_NULL


def test_rmsnorm_argument_validation_needs_no_device(lib):
    A, MB = 0x10000, 1 << 20
    H, G, Z = A, A + 64 * MB, A + 128 * MB
    f = lib.kx_rmsnorm
    assert f(H, G, 1e-6, Z, 4, 12, None) == kx.KX_ERR_SHAPE          # N % 8
    assert f(H, G, 1e-6, Z, 4, 32768 + 8, None) == kx.KX_ERR_SHAPE   # row too long for one CTA
    assert f(H, G, -1.0, Z, 4, 8, None) == kx.KX_ERR_SHAPE           # eps < 0
    assert f(H, G, float("nan"), Z, 4, 8, None) == kx.KX_ERR_SHAPE
    assert f(None, G, 1e-6, Z, 4, 8, None) == kx.KX_ERR_NULL
    assert f(H, G + 2, 1e-6, Z, 4, 8, None) == kx.KX_ERR_ALIGN
    assert f(H, G, 1e-6, H + 16, 4, 8, None) == kx.KX_ERR_OVERLAP    # partial overlap with H
    assert f(H, G, 1e-6, G, 4, 8, None) == kx.KX_ERR_OVERLAP
    assert f(None, None, 1e-6, None, 0, 8, None) == kx.KX_OK
    g = lib.kx_outproj_residual_rmsnorm
    X, W, R = A + 192 * MB, A + 256 * MB, A + 320 * MB
    assert g(X, W, None, R, G, 1e-6, H, H, 4, 8, 8, None) == kx.KX_ERR_OVERLAP   # Z == H
    assert g(X, W, None, R, G, 1e-6, H, X, 4, 8, 8, None) == kx.KX_ERR_OVERLAP
    assert g(X, W, None, None, G, 1e-6, H, Z, 4, 8, 8, None) == kx.KX_ERR_NULL   # residual required
    assert g(X, W, None, R, G, 1e-6, H, Z, 4, 8, 12, None) == kx.KX_ERR_SHAPE


def test_binding_rejects_wrong_tensors():
    import torch
    X = torch.zeros(4, 8, dtype=torch.float32)
    W = torch.zeros(8, 8, dtype=torch.bfloat16)
    Y = torch.zeros(4, 8, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        kx.kx_gemm_bf16(X, W, Y, stream=0)
    with pytest.raises(ValueError):
        kx.kx_gemm_bf16(W[:4].t(), W, Y, stream=0)
    with pytest.raises(TypeError):
        kx.make_override(bogus=1)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(kx, "_lib", None)
    monkeypatch.setattr(kx, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        kx.load()


def test_product_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_2608_17071_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", text, flags=re.M), fn
                assert "kx_oracle" not in text, fn


def test_bound_call_keeps_its_tensors_alive(lib):
    """The pre-marshalled callable stores raw addresses, so it must own references
    to the tensors: otherwise their memory could be released while calls remain."""
    import gc
    import weakref
    import torch
    X = torch.zeros(4, 8, dtype=torch.bfloat16)
    W = torch.zeros(8, 8, dtype=torch.bfloat16)
    R = torch.zeros(4, 8, dtype=torch.bfloat16)
    Y = torch.zeros(4, 8, dtype=torch.bfloat16)
    refs = [weakref.ref(t) for t in (X, W, R, Y)]
    f = kx.bound_call(X, W, None, R, Y, stream=0)
    del X, W, R, Y
    gc.collect()
    assert all(r() is not None for r in refs)
    assert len(f.tensors) == 7
    del f
    gc.collect()
    assert all(r() is None for r in refs)
