"""Builds libminicache.so (sm_100a) in-tree with nvcc.  `python -m paper_2405_14366_b200.build`."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libminicache.so")
BOUNDS_LIB_PATH = os.path.join(PKG_DIR, "libminicache_bounds.so")  # the range-checked build (-DMC_BOUNDS=1)
SOURCES = ["mc_api.cu", "mc_merge.cu", "mc_restore.cu", "mc_attn.cu", "mc_q4cache.cu", "mc_prefill.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, bounds: bool = False) -> str:
    """Compile every kernel file and link the shared library; returns its path.
    bounds: the range-checked build (every kernel compiled with -DMC_BOUNDS=1) as libminicache_bounds.so."""
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(ROOT, "include", "minicache.h"))
    headers.append(os.path.abspath(__file__))  # flag changes rebuild everything
    objs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(CSRC, src.replace(".cu", ".bounds.o" if bounds else ".o"))
        objs.append(o)
        if force or _stale(o, [s] + headers):
            cmd = [_nvcc()] + NVCC_FLAGS + (["-DMC_BOUNDS=1"] if bounds else []) + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            subprocess.run(cmd, check=True)
    lib_path = BOUNDS_LIB_PATH if bounds else LIB_PATH
    if force or _stale(lib_path, objs):
        cmd = [_nvcc(), "-shared", "-o", lib_path] + objs + ["-gencode", "arch=compute_100a,code=sm_100a", "-ldl"]
        subprocess.run(cmd, check=True)
    return lib_path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, bounds="--bounds" in sys.argv))
