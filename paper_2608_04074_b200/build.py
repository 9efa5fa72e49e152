"""In-tree builds: the CUDA C-ABI library (nvcc, sm_100a) and the host calibration helper (gcc).

Artefacts are written next to this file so that they travel with a snapshot of the tree.
"""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

PKG_DIR = Path(__file__).resolve().parent
CSRC = PKG_DIR / "csrc"
INCLUDE = PKG_DIR.parent / "include"
LIB_CUDA = PKG_DIR / "libnovakv.so"
LIB_CALIB = PKG_DIR / "libnovakv_calib.so"

CUDA_SOURCES = ["novakv_api.cu", "novakv_encode.cu", "novakv_decode.cu", "novakv_bf16_decode.cu",
                "novakv_noalloc.cu"]


def _newer(target: Path, sources: list[Path]) -> bool:
    if not target.exists():
        return False
    t = target.stat().st_mtime
    return all(s.stat().st_mtime <= t for s in sources)


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def build_cuda(force: bool = False, verbose: bool = False) -> Path:
    srcs = [CSRC / s for s in CUDA_SOURCES if (CSRC / s).exists()]
    deps = srcs + sorted(CSRC.glob("*.cuh")) + sorted(INCLUDE.glob("*.h"))
    if not force and _newer(LIB_CUDA, deps):
        return LIB_CUDA
    cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
           "-std=c++17", "-Xcompiler", "-fPIC", "-I", str(INCLUDE), "-I", str(CSRC)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [str(s) for s in srcs] + ["-o", str(LIB_CUDA)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return LIB_CUDA


def build_calib_host(force: bool = False) -> Path:
    src = CSRC / "calib_host.c"
    if not force and _newer(LIB_CALIB, [src]):
        return LIB_CALIB
    cmd = ["gcc", "-O3", "-fopenmp", "-shared", "-fPIC", str(src), "-o", str(LIB_CALIB)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("gcc failed:\n" + res.stdout + res.stderr)
    return LIB_CALIB
