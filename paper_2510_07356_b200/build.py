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


def _compile(lib: Path, srcs, verbose: bool) -> None:
    tmp = lib.with_suffix(f".{os.getpid()}.tmp")
    cmd = [_nvcc(), *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", str(tmp), *map(str, srcs)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)


def build_bench(force: bool = False, verbose: bool = False) -> Path:
    """The benchmark's helper library: one kernel, nothing of the attention path."""
    srcs = sorted(BENCH_CSRC.glob("*.cu"))
    deps = srcs + list(BENCH_CSRC.glob("*.h"))
    if force or not BENCH_LIB.exists() or any(d.stat().st_mtime > BENCH_LIB.stat().st_mtime for d in deps):
        _compile(BENCH_LIB, srcs, verbose)
    return BENCH_LIB


def build(force: bool = False, verbose: bool = False) -> Path:
    build_bench(force, verbose)
    if not force and not needs_build():
        return LIB
    _compile(LIB, sources(), verbose)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
