"""Builds the CUDA library in-tree: `nvcc` cross-compiles csrc/hisparse.cu (which includes the other files of
csrc/) for sm_100a into `_hisparse.so` next to this file (no GPU needed to build)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
SRC = os.path.join(_HERE, "csrc", "hisparse.cu")
HEADER = os.path.join(ROOT, "include", "hisparse.h")
SO = os.path.join(_HERE, "_hisparse.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def needs_build() -> bool:
    if not os.path.exists(SO):
        return True
    t = os.path.getmtime(SO)
    csrc = os.path.dirname(SRC)          # hisparse.cu includes the other files of csrc/: one translation unit
    deps = [os.path.join(csrc, f) for f in os.listdir(csrc)] + [HEADER]
    return any(os.path.getmtime(p) > t for p in deps)


def build_cuda(force: bool = False, verbose: bool = False) -> str:
    if force or needs_build():
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = SO + ".tmp%d" % os.getpid()
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
              ["-I", os.path.join(ROOT, "include"), "-o", tmp, SRC]
        subprocess.check_call(cmd)
        os.replace(tmp, SO)
    return SO


if __name__ == "__main__":
    print(build_cuda(force=True, verbose=True))
