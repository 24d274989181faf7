"""Builds libkvsink.so (hand-written CUDA for sm_100a) in-tree with nvcc.

Every translation unit is compiled to an object of its own (in parallel, only when it is older than its sources) and
the objects are linked into the shared library; no kernel calls device code of another unit, so no device link step
is needed.
"""
from __future__ import annotations

import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libkvsink.so")
HEADER = os.path.join(os.path.dirname(HERE), "include", "kvsink.h")
SOURCES = ["api.cu", "predict.cu", "quantize.cu", "quantize_groups.cu", "quantize_bulk.cu", "decode.cu", "decode_b2.cu", "decode_b3.cu", "decode_b4.cu", "analysis.cu", "calibrated.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC"]


def _headers():
    return [HEADER] + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]


def _older(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


DEBUG_LIB = os.path.join(HERE, "libkvsink_debug.so")


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles what is stale and returns the library's path.  debug=True builds libkvsink_debug.so with -DKVSINK_DEBUG:
    the same kernels with index checks that raise KVSINK_STATUS_BOUNDS instead of touching memory outside an array."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    OBJ = os.path.join(HERE, "_build_debug" if debug else "_build")
    LIB = DEBUG_LIB if debug else globals()["LIB"]
    defines = ("KVSINK_DEBUG",) if debug else ()
    os.makedirs(OBJ, exist_ok=True)
    hdrs = _headers()
    jobs = []
    for s in SOURCES:
        src, obj = os.path.join(CSRC, s), os.path.join(OBJ, s[:-3] + ".o")
        if force or _older(obj, [src] + hdrs):
            cmd = [nvcc] + NVCC_FLAGS + [f"-D{d}" for d in defines] + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            jobs.append((s, obj, cmd))

    def run(job):
        s, obj, cmd = job
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0 and os.path.exists(obj):
            os.remove(obj)
        return s, r

    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as ex:
            results = list(ex.map(run, jobs))
        for s, r in results:
            if verbose or r.returncode != 0:
                print(f"---- {s}\n{r.stdout}{r.stderr}", flush=True)
        bad = [s for s, r in results if r.returncode != 0]
        if bad:
            if os.path.exists(LIB):
                os.remove(LIB)      # never leave a stale library behind a failed build
            raise RuntimeError(f"nvcc failed on {', '.join(bad)}")
    objs = [os.path.join(OBJ, s[:-3] + ".o") for s in SOURCES]
    if jobs or _older(LIB, objs):
        r = subprocess.run([nvcc, "-shared", "-o", LIB] + objs)
        if r.returncode != 0:
            if os.path.exists(LIB):
                os.remove(LIB)
            raise RuntimeError(f"link failed with status {r.returncode}")
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="-f" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
