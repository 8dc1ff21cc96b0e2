"""Build libkx.so (the C-ABI CUDA library) in-tree for sm_100a.

``python -m paper_2608_17071_b200.build`` or ``build()``.  nvcc cross-compiles
without a GPU.  Every ``.cu`` file under ``csrc/`` is one translation unit, compiled to an
object file of its own (in parallel, rebuilt only when it or a header changed) and linked
into one shared library.  The library links the static CUDA runtime, so it loads on a
machine without a driver (argument validation still works there).
"""
from __future__ import annotations

import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libkx.so")
SOURCES = ["kx_api.cu", "kx_gemv.cu", "kx_rowcode.cu"]
HEADERS = ["kx_kernels.cuh", "kx_ptx.cuh", "kx_gemv.cuh", "kx_rowcode.cuh", "kx_internal.h", "kx_plan_table.inc",
           os.path.join("..", "..", "include", "kx.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _newest_header() -> float:
    return max(os.path.getmtime(os.path.join(CSRC, h)) for h in HEADERS)


def _obj(src: str) -> str:
    return os.path.join(OBJ, os.path.splitext(src)[0] + ".o")


def _obj_stale(src: str) -> bool:
    o = _obj(src)
    if not os.path.exists(o):
        return True
    t = os.path.getmtime(o)
    return os.path.getmtime(os.path.join(CSRC, src)) > t or _newest_header() > t


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, s)) > t for s in SOURCES) or _newest_header() > t


def _compile(src: str, verbose: bool) -> None:
    cmd = [_nvcc(), *NVCC_FLAGS]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    tmp = _obj(src) + f".tmp{os.getpid()}"
    cmd += ["-c", os.path.join(CSRC, src), "-o", tmp]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _obj(src))


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    todo = [s for s in SOURCES if force or _obj_stale(s)]
    with ThreadPoolExecutor(max_workers=max(1, len(todo))) as ex:
        list(ex.map(lambda s: _compile(s, verbose), todo))
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.run([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + [_obj(s) for s in SOURCES], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
