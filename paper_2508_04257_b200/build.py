"""Builds libkvsink.so (hand-written CUDA for sm_100a) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libkvsink.so")
SOURCES = ["api.cu", "predict.cu", "quantize.cu", "quantize_groups.cu", "quantize_bulk.cu", "decode.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-shared", "-Xcompiler", "-fPIC"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(os.path.dirname(HERE), "include", "kvsink.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
        r = subprocess.run(cmd)
        if r.returncode != 0:
            if os.path.exists(LIB):
                os.remove(LIB)      # never leave a stale library behind a failed build
            raise RuntimeError(f"nvcc failed with status {r.returncode}")
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
