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


def _deps_mtime() -> float:
    hdrs = list(CSRC.glob("*.cuh")) + [PKG.parent / "include" / "hawk.h"]
    return max(h.stat().st_mtime for h in hdrs)


def _flags(verbose: bool, extra=()):
    flags = ["-std=c++17", "-O3", "-lineinfo", *ARCH_FLAGS, "-Xcompiler", "-fPIC"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    flags += list(extra)
    return flags + os.environ.get("HAWK_NVCC_FLAGS", "").split()   # e.g. -DHAWK_ATTN_WARPS=4 -DHAWK_ATTN_STAGE_KB=16


def build(force: bool = False, verbose: bool = False, lib: Path = LIB, objdir: Path | None = None,
          extra_flags=()) -> Path:
    """Compiles every source to an object of its own (in parallel; only the ones whose source or headers changed)
    and links them into `lib`."""
    objdir = objdir or (PKG / "_build")
    objdir.mkdir(exist_ok=True)
    tag = objdir / "flags.txt"
    flags = _flags(verbose, extra_flags)
    if not tag.exists() or tag.read_text() != " ".join(flags):
        force = True
    hdr_t = _deps_mtime()
    jobs = []
    for src in SOURCES:
        obj = objdir / (Path(src).stem + ".o")
        s = CSRC / src
        if force or not obj.exists() or obj.stat().st_mtime < max(s.stat().st_mtime, hdr_t):
            jobs.append((s, obj))
    if not jobs and lib.exists() and all(lib.stat().st_mtime >= (objdir / (Path(s).stem + ".o")).stat().st_mtime
                                         for s in SOURCES):
        return lib
    nvcc = _nvcc()

    def compile_one(job):
        s, obj = job
        return s, subprocess.run([nvcc, *flags, "-c", str(s), "-o", str(obj)], capture_output=True, text=True)

    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as pool:
        for s, res in pool.map(compile_one, jobs):
            if res.returncode != 0:
                sys.stderr.write(res.stdout + res.stderr)
                raise RuntimeError(f"nvcc failed on {s.name}")
            if verbose:
                sys.stderr.write(res.stderr)
    tag.write_text(" ".join(flags))
    tmp = lib.with_suffix(f".{os.getpid()}.tmp")
    objs = [str(objdir / (Path(s).stem + ".o")) for s in SOURCES]
    res = subprocess.run([nvcc, *ARCH_FLAGS, "-shared", "-cudart", "static", "-o", str(tmp), *objs],
                         capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed linking " + lib.name)
    os.replace(tmp, lib)
    return lib


STALL_LIB = PKG / "libhawk_verify_stall.so"


def build_stall_variant(force: bool = False) -> Path:
    """The library the give-up tests load: every wait limited to 2 ms, and one stage per kernel armed for more
    bytes than its copies deliver (HAWK_TEST_STALL), so that exactly one wait per launch runs out."""
    return build(force=force, lib=STALL_LIB, objdir=PKG / "_build_stall",
                 extra_flags=("-DHAWK_WAIT_NS=2000000ull", "-DHAWK_TEST_STALL"))


DEBUG_LIB = PKG / "libhawk_verify_debug.so"


def build_debug_variant(force: bool = False) -> Path:
    """The library with index checks compiled in (-DHAWK_DEBUG): every checked index that leaves its array raises
    HAWK_DEV_BOUNDS in the call's status word and the access is skipped.  The stand-in for a memory checker."""
    return build(force=force, lib=DEBUG_LIB, objdir=PKG / "_build_debug", extra_flags=("-DHAWK_DEBUG",))


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
