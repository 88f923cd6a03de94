"""Build step: compile the CUDA sources under ``csrc/`` into ``libcpattn.so`` (sm_100a only).

The library is built in-tree next to this file with plain ``nvcc`` (which cross-compiles without a
GPU).  ``python -m paper_2609_04774_b200.build`` rebuilds it.
"""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libcpattn.so")
SOURCES = ["ctx.cu", "plan.cpp", "cache_manager.cpp", "merge.cu", "kv_copy.cu", "attn_sm100.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every source to an object in ``build/`` and link ``libcpattn.so``.  Returns its path."""
    headers = [os.path.join(CSRC, "internal.h"), os.path.join(CSRC, "attn_kernel.cuh"), os.path.join(ROOT, "include", "cpattn.h"),
               os.path.join(ROOT, "include", "cpcache.h"), os.path.abspath(__file__)]
    objdir = os.path.join(_HERE, "build")
    os.makedirs(objdir, exist_ok=True)
    objs = []
    for src in SOURCES:
        sp = os.path.join(CSRC, src)
        obj = os.path.join(objdir, os.path.splitext(src)[0] + ".o")
        objs.append(obj)
        if force or _stale(obj, [sp] + headers):
            cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", sp, "-o", obj]
            subprocess.check_call(cmd)
    if force or _stale(LIB_PATH, objs):
        subprocess.check_call([_nvcc(), "-shared", "-o", LIB_PATH] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
