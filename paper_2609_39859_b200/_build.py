"""Builds libfork_dllm.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libfork_dllm.so")
SOURCES = ["fork_dllm.cu"]
HEADERS = ["fork_partition.h", "fork_reduce.cuh", "fork_params.cuh", "fork_setup.cuh", "fork_finalize.cuh", "fork_stream.cuh", "fork_head.cuh"]


def sources():
    return [os.path.join(CSRC, s) for s in SOURCES]


def _deps():
    return sources() + [os.path.join(CSRC, h) for h in HEADERS] + [os.path.join(_ROOT, "include", "fork_dllm.h")]


def nvcc_command(out: str, extra=()):
    return ["nvcc", "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
            "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include"), *extra, "-o", out, *sources()]


def build(force: bool = False, verbose: bool = False) -> str:
    stale = force or not os.path.exists(LIB) or any(os.path.getmtime(LIB) < os.path.getmtime(d) for d in _deps())
    if stale:
        tmp = LIB + ".tmp%d" % os.getpid()
        cmd = nvcc_command(tmp, ("-Xptxas", "-v") if verbose else ())
        subprocess.check_call(cmd)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
