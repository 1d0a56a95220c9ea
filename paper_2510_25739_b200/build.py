"""Builds the C-ABI shared library (libhawk_verify.so) in-tree with nvcc for sm_100a.

nvcc cross-compiles without a GPU.  The library links the CUDA runtime statically and reaches the
one driver call it needs (tensor-map encoding) through the runtime's driver entry point.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libhawk_verify.so"
SOURCES = ["hawk_api.cu", "hawk_accept.cu", "hawk_attn.cu", "hawk_head.cu", "hawk_step.cu", "hawk_pool.cu"]
ARCH_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not Path(exe).exists():
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + [PKG.parent / "include" / "hawk.h"]
    return any(d.stat().st_mtime > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not _stale():
        return LIB
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
    cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", *ARCH_FLAGS, "-Xcompiler", "-fPIC", "-shared",
           "-cudart", "static", "-o", str(tmp)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += os.environ.get("HAWK_NVCC_FLAGS", "").split()   # e.g. -DHAWK_ATTN_WARPS=4 -DHAWK_ATTN_STAGE_KB=16
    cmd += [str(CSRC / s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libhawk_verify.so")
    if verbose:
        sys.stderr.write(res.stderr)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
