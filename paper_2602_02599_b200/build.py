"""Builds the C-ABI shared library in-tree with nvcc for sm_100a (no JIT cache, no torch headers)."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "librap_b200.so")
OBJ = os.path.join(HERE, "_build")
SOURCES = ["rap_api.cu", "rap_proj.cu", "rap_proj_tc.cu", "rap_attn.cu", "rap_attn_fast.cu", "rap_attn_scan.cu",
           "rap_lowrank.cu", "rap_lowrank_tc.cu"]


def _stale():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "rap.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False):
    """Compile every CUDA source into librap_b200.so; returns the library path."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
             "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    os.makedirs(OBJ, exist_ok=True)

    def compile_one(src):
        obj = os.path.join(OBJ, src.replace(".cu", ".o"))
        path = os.path.join(CSRC, src)
        deps = [path, os.path.join(CSRC, "rap_internal.h"), os.path.join(INCLUDE, "rap.h")]
        if not force and os.path.exists(obj) and all(os.path.getmtime(d) <= os.path.getmtime(obj) for d in deps):
            return obj, None
        return obj, subprocess.run([nvcc] + flags + ["-c", path, "-o", obj], capture_output=True, text=True)

    with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:     # one nvcc process per translation unit
        results = list(pool.map(compile_one, SOURCES))
    for obj, res in results:
        if res is not None and (verbose or res.returncode):
            sys.stderr.write(res.stdout + res.stderr)
        if res is not None and res.returncode:
            raise RuntimeError("nvcc failed compiling " + obj)
    res = subprocess.run([nvcc, "-shared", "-o", LIB] + [o for o, _ in results], capture_output=True, text=True)
    if res.returncode:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed linking librap_b200.so")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
