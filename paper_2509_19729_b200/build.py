"""Builds the CUDA library in-tree: ``python -m paper_2509_19729_b200.build``.

nvcc cross-compiles for sm_100a without a GPU.  The shared object lands next to this file so that it travels
with the source tree; nothing is installed into site-packages and nothing is JIT-cached elsewhere.
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
INCLUDE = HERE.parent / "include"
LIB = HERE / "libamoeba.so"
LIB_CHECKED = HERE / "libamoeba_checked.so"  # the same sources with -DAMOEBA_CHECK_ITEMS: every work item is tested
#                                              against the extent of its buffers before it is moved
SOURCES = ["plan.cpp", "block_tables.cu", "kv_reshard.cu", "weights_reshard.cu"]
HEADERS = ["plan.hpp", "launch.hpp", "copy_engine.cuh", "kv_items.cuh", "w_items.cuh"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
    "-Xcompiler", "-fvisibility=hidden", "-shared", "-cudart", "static",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build(checked: bool = False) -> bool:
    lib = LIB_CHECKED if checked else LIB
    if not lib.exists():
        return True
    t = lib.stat().st_mtime
    deps = [CSRC / s for s in SOURCES + HEADERS] + [INCLUDE / "amoeba.h"]
    return any(d.stat().st_mtime > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> Path:
    lib = LIB_CHECKED if checked else LIB
    if not force and not needs_build(checked):
        return lib
    tmp = lib.with_suffix(f".tmp{os.getpid()}.so")
    cmd = [_nvcc(), *NVCC_FLAGS, f"-I{INCLUDE}", f"-I{CSRC}"]
    if checked:
        cmd += ["-DAMOEBA_CHECK_ITEMS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [str(CSRC / s) for s in SOURCES] + ["-o", str(tmp)]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
