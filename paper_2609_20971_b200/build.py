"""Builds the C-ABI CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "librbs_b200.so")
LIB_DEBUG = os.path.join(PKG, "librbs_b200_debug.so")   # the same sources with -DRBS_DEBUG: device-side index checks
SOURCES = ["rbs_api.cu", "rbs_tmap.cu", "rbs_stats.cu", "rbs_select.cu", "rbs_prefill.cu", "rbs_prefill_pair.cu", "rbs_union.cu", "rbs_box.cu", "rbs_varlen.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if not f.endswith(".o")]
    deps += [os.path.join(ROOT, "include", "rbs.h"), os.path.join(ROOT, "include", "rbs_selftest.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles the sources (in parallel) and links the library; debug=True builds the checking variant."""
    from concurrent.futures import ThreadPoolExecutor

    lib = LIB_DEBUG if debug else LIB
    if not force and not needs_build(lib):
        return lib
    suffix = ".debug.o" if debug else ".o"
    extra = ["-DRBS_DEBUG"] if debug else []

    def compile_one(src: str) -> str:
        obj = os.path.join(CSRC, src.replace(".cu", suffix))
        cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c",
               os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        subprocess.run(cmd, check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    subprocess.run([_nvcc(), "-shared", "-o", lib, *objs, "-lcudart_static", "-ldl", "-lrt", "-lpthread"], check=True)
    return lib


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
