"""Builds libconcur_attn.so (the attention library) and libconcur_bench.so (the benchmark's read-only
stream probe) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libconcur_attn.so"
BOUNDS_LIB = PKG / "libconcur_attn_bounds.so"
BENCH_CSRC = PKG / "bench_csrc"
BENCH_LIB = PKG / "libconcur_bench.so"
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--use_fast_math", "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def _nvcc() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return cand


def sources():
    return sorted(CSRC.glob("*.cu"))


def needs_build() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list((PKG.parent / "include").glob("*.h"))
    return any(d.stat().st_mtime > t for d in deps)


def _compile(lib: Path, srcs, verbose: bool, defines=()) -> None:
    tmp = lib.with_suffix(f".{os.getpid()}.tmp")
    cmd = [_nvcc(), *NVCC_FLAGS, *defines, *(["-Xptxas", "-v"] if verbose else []), "-o", str(tmp), *map(str, srcs)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)


def build_bench(force: bool = False, verbose: bool = False) -> Path:
    """The benchmark's helper library: one kernel, nothing of the attention path."""
    srcs = sorted(BENCH_CSRC.glob("*.cu"))
    deps = srcs + list(BENCH_CSRC.glob("*.h"))
    if force or not BENCH_LIB.exists() or any(d.stat().st_mtime > BENCH_LIB.stat().st_mtime for d in deps):
        _compile(BENCH_LIB, srcs, verbose)
    return BENCH_LIB


def build_bounds(force: bool = False, verbose: bool = False) -> Path:
    """The checked build: the same sources with -DCONCUR_BOUNDS, in which every index the kernels compute
    for the workspace, the partial buffers and the outputs is held against its buffer's capacity
    (a violation is recorded as CONCUR_FLAG_BOUNDS and the access skipped).  Load it by setting
    CONCUR_ATTN_LIBRARY to its path before importing the package."""
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list((PKG.parent / "include").glob("*.h"))
    if force or not BOUNDS_LIB.exists() or any(d.stat().st_mtime > BOUNDS_LIB.stat().st_mtime for d in deps):
        _compile(BOUNDS_LIB, sources(), verbose, ("-DCONCUR_BOUNDS",))
    return BOUNDS_LIB


def build(force: bool = False, verbose: bool = False) -> Path:
    build_bench(force, verbose)
    if not force and not needs_build():
        return LIB
    _compile(LIB, sources(), verbose)
    return LIB


if __name__ == "__main__":
    import sys
    if "--bounds" in sys.argv:
        print(build_bounds(force=True, verbose="-v" in sys.argv))
    else:
        print(build(force=True, verbose="-v" in sys.argv))
