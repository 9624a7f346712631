"""Builds the C-ABI shared library (liblibra.so) in-tree with nvcc for sm_100a.

nvcc cross-compiles without a GPU, so this also runs on a CPU-only machine.  The CUDA runtime is
linked statically and the driver API is reached through the runtime's entry-point lookup, so the
library loads on machines without a driver (the planner entry point needs no GPU).
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB_PATH = os.path.join(HERE, "liblibra.so")
STAMP_PATH = os.path.join(HERE, "liblibra.so.stamp")

SOURCES = ["libra_api.cu", "planner.cpp", "sched.cpp", "ring_sched.cpp"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--use_fast_math", "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _source_digest(extra_flags) -> str:
    h = hashlib.sha256()
    names = sorted(os.listdir(CSRC)) + [os.path.join(INCLUDE, "libra.h")]
    for n in names:
        path = n if os.path.isabs(n) else os.path.join(CSRC, n)
        with open(path, "rb") as f:
            h.update(n.encode() + b"\0" + f.read())
    h.update(" ".join(NVCC_FLAGS + list(extra_flags)).encode())
    return h.hexdigest()


def build_library(force: bool = False, verbose: bool = True, extra_flags=()) -> str:
    """Compile if the sources changed since the last build; returns the library path."""
    digest = _source_digest(extra_flags)
    if not force and os.path.exists(LIB_PATH) and os.path.exists(STAMP_PATH):
        with open(STAMP_PATH) as f:
            if f.read().strip() == digest:
                return LIB_PATH
    cmd = [_nvcc(), *NVCC_FLAGS, *extra_flags, "-I", INCLUDE, "-I", CSRC,
           *[os.path.join(CSRC, s) for s in SOURCES], "-o", LIB_PATH]
    if verbose:
        print(" ".join(cmd), flush=True)
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed")
    with open(STAMP_PATH, "w") as f:
        f.write(digest)
    return LIB_PATH


if __name__ == "__main__":
    build_library(force="--force" in sys.argv, extra_flags=[a for a in sys.argv[1:] if a.startswith(("-X", "-D"))])
