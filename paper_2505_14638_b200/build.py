"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libw4a8_b200.so")
SOURCES = [os.path.join(CSRC, "w4a8_lib.cu")]


def _deps():
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(_HERE), "include", "w4a8.h"))
    return deps


def nvcc_command(out_path: str, verbose: bool = False):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [
        nvcc, "-std=c++17", "-O3", "-lineinfo",
        "-gencode", "arch=compute_100a,code=sm_100a",
        "-Xcompiler", "-fPIC", "-shared",
        "-o", out_path,
    ]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    return cmd + SOURCES + ["-lcudart"]


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile when the library is missing or older than a source. Returns the .so path."""
    stale = force or not os.path.exists(LIB_PATH) or any(
        os.path.getmtime(d) > os.path.getmtime(LIB_PATH) for d in _deps())
    if stale:
        tmp = LIB_PATH + ".tmp%d" % os.getpid()
        res = subprocess.run(nvcc_command(tmp, verbose), capture_output=True, text=True)
        if verbose:
            sys.stderr.write(res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
