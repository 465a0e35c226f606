"""In-tree build of libkangaroo.so with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc")
_OUT = os.path.join(_HERE, "libkangaroo.so")
_SOURCES = ["kg_api.cu"]
_DEPS = ["kg_api.cu", "kg_engine.cuh", "kg_device.cuh", "kg_prefill.cuh", os.path.join("..", "..", "include", "kangaroo.h")]


def lib_path() -> str:
    return _OUT


def _stale() -> bool:
    if not os.path.exists(_OUT):
        return True
    t = os.path.getmtime(_OUT)
    return any(os.path.getmtime(os.path.join(_SRC, d)) > t for d in _DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return _OUT
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", _OUT] + [os.path.join(_SRC, s) for s in _SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + r.stdout + r.stderr)
    if verbose:
        print(r.stderr)
    return _OUT
