"""Builds the CUDA library in-tree for sm_100a with nvcc (no JIT cache, no torch extension machinery).

Every source is compiled to an object file of its own (in parallel, only when it or a header changed) and the
objects are linked into libsketched_amsgrad.so beside this file.  SK_NVCC_EXTRA adds flags (e.g. -DSK_DEBUG=1).
"""
from __future__ import annotations

import concurrent.futures
import hashlib
import os
import shlex
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libsketched_amsgrad.so")
LIB_DEBUG = os.path.join(HERE, "libsketched_amsgrad_debug.so")    # device-side bounds checks compiled in
SOURCES = ["sk_api.cu", "sk_sketch.cu", "sk_sketch_own.cu", "sk_select.cu", "sk_static.cu", "sk_shard.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _flags(verbose: bool, debug: bool = False) -> list[str]:
    flags = list(NVCC_FLAGS) + shlex.split(os.environ.get("SK_NVCC_EXTRA", ""))
    if debug:
        flags += ["-DSK_DEBUG=1"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    return flags


def _headers() -> list[str]:
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if not f.endswith(".cu")]
    hs.append(os.path.join(os.path.dirname(HERE), "include", "sketched_amsgrad.h"))
    return hs


def _object(src: str, flags: list[str]) -> str:
    tag = hashlib.sha256(" ".join(flags).encode()).hexdigest()[:10]
    return os.path.join(OBJ, f"{os.path.splitext(src)[0]}.{tag}.o")


def _compile(src: str, flags: list[str], force: bool) -> str:
    obj = _object(src, flags)
    path = os.path.join(CSRC, src)
    deps = [path] + _headers()
    if force or not os.path.exists(obj) or any(os.path.getmtime(p) > os.path.getmtime(obj) for p in deps):
        tmp = obj + f".{os.getpid()}.tmp"
        subprocess.run([_nvcc()] + flags + ["-c", "-o", tmp, path], check=True)
        os.replace(tmp, obj)
    return obj


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds (if stale) and returns the library's path; debug=True builds the bounds-checked variant beside it."""
    flags = _flags(verbose, debug)
    LIB = LIB_DEBUG if debug else globals()["LIB"]
    os.makedirs(OBJ, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(lambda s: _compile(s, flags, force), SOURCES))
    if force or not os.path.exists(LIB) or any(os.path.getmtime(o) > os.path.getmtime(LIB) for o in objs):
        tmp = LIB + f".{os.getpid()}.tmp"
        subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs, check=True)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
