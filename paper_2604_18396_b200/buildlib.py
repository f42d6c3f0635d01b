"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU).

One object per translation unit, compiled in parallel, linked into libriver_b200.so next to this file.
"""
from __future__ import annotations

import concurrent.futures
import os
import shlex
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
OBJ = os.path.join(_HERE, "build")
LIB = os.path.join(_HERE, "libriver_b200.so")
SOURCES = ["river_api.cu", "launch_stream.cu", "launch_attn.cu", "launch_tc.cu", "launch_tc_w4.cu", "noalloc_argmax.cu", "quantize_w4.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _deps():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_HERE, "..", "include", "river.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libriver_b200.so; returns its path.  NVCC names the compiler, NVCC_EXTRA adds flags."""
    if not (force or _stale()):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    extra = shlex.split(os.environ.get("NVCC_EXTRA", ""))
    os.makedirs(OBJ, exist_ok=True)
    newest_hdr = max(os.path.getmtime(d) for d in _deps() if not d.endswith(".cu"))

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ, src[:-3] + ".o")
        path = os.path.join(CSRC, src)
        if not force and not extra and os.path.exists(obj) and os.path.getmtime(obj) > max(newest_hdr, os.path.getmtime(path)):
            return obj
        cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", path, "-o", obj]
        if verbose:
            print(" ".join(cmd))
        subprocess.check_call(cmd)
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    subprocess.check_call([nvcc, "-shared"] + NVCC_FLAGS[:2] + ["-o", LIB] + objs)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
