"""Builds the C-ABI shared library (libverillm.so) in-tree with nvcc for sm_100a.

    python -m paper_2509_24257_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU.  Objects go to _build/ inside the package (not committed).
"""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
BUILD = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libverillm.so")
SOURCES = ["gemm_tcgen05.cu", "attention_tcgen05.cu", "elementwise.cu", "merkle.cu", "verillm.cu"]
HEADERS = ["common.cuh", "compare.cuh", "kernels.h", os.path.join("..", "..", "include", "verillm.h")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr",
]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _newest(paths) -> float:
    return max(os.path.getmtime(p) for p in paths)


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return _newest(deps) > os.path.getmtime(LIB)


def build_library(force: bool = False, verbose: bool = False, defines=(), out: str | None = None) -> str:
    """Compiles and links the library.  `defines` (-D macros) and `out` build a tuning variant elsewhere."""
    variant = bool(defines) or out is not None
    lib_path = out or LIB
    if not variant and not force and not is_stale():
        return LIB
    build_dir = BUILD if not variant else os.path.join(BUILD, "variant_" + os.path.basename(lib_path))
    os.makedirs(build_dir, exist_ok=True)
    extra = (["-Xptxas", "-v"] if verbose else []) + [f"-D{d}" for d in defines]

    def compile_one(src: str) -> str:
        obj = os.path.join(build_dir, src.replace(".cu", ".o"))
        cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib_path, *objs]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("link failed")
    return lib_path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
