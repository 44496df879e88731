"""Builds the CUDA library (``libhikonv.so``) for sm_100a with nvcc, in-tree.

Every translation unit under ``csrc/`` is compiled to an object under ``_build/`` (only when it or a header is
newer than the object), side by side, and the objects are linked into one shared library.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(HERE, "libhikonv.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-lineinfo", "-std=c++17", "--use_fast_math",
    "-Xcompiler", "-fPIC",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cpp")))


def _headers():
    return (glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh"))
            + glob.glob(os.path.join(ROOT, "include", "*.h")))


def _object_of(src: str) -> str:
    return os.path.join(OBJ_DIR, os.path.basename(src) + ".o")


def build(force: bool = False, verbose: bool = False, extra_flags=()) -> str:
    """Compile what is out of date under csrc/ and link the shared library; a no-op when nothing changed."""
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    newest_header = max(os.path.getmtime(h) for h in _headers())
    flags = NVCC_FLAGS + list(extra_flags) + ["-I", os.path.join(ROOT, "include"), "-I", CSRC]
    stale = [s for s in sources()
             if force or extra_flags or not os.path.exists(_object_of(s))
             or os.path.getmtime(_object_of(s)) < max(os.path.getmtime(s), newest_header)]

    def compile_one(src: str) -> None:
        cmd = [nvcc] + flags + ["-c", src, "-o", _object_of(src)]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)

    if stale:
        with ThreadPoolExecutor(max_workers=min(len(stale), os.cpu_count() or 4)) as pool:
            list(pool.map(compile_one, stale))
    objects = [_object_of(s) for s in sources()]
    if stale or not os.path.exists(LIB_PATH) or os.path.getmtime(LIB_PATH) < max(os.path.getmtime(o) for o in objects):
        tmp = LIB_PATH + ".tmp.%d" % os.getpid()
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objects
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    flags = ["-Xptxas", "-v"] if "--ptxas" in sys.argv else []
    print(build(force="--force" in sys.argv, verbose=True, extra_flags=flags))
