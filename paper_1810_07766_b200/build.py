"""Builds ``csrc/librps.so`` in-tree with nvcc for sm_100a (no GPU needed to compile)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(CSRC, "librps.so")
SOURCES = ["rps_api.cu", "rps_kernels.cu", "rps_static.cu"]
HEADERS = ["rps_device.cuh", "rps_kernels.h"]


def nvcc_command(out: str = LIB, extra=()):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    return [nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
            "-Xcompiler", "-fPIC,-Wall", "-shared", "-cudart", "static", "-I", INCLUDE, "-I", CSRC,
            *extra, "-o", out, *[os.path.join(CSRC, s) for s in SOURCES]]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(INCLUDE, "rps.h")]
    return any(os.path.getmtime(f) > built for f in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or is_stale():
        tmp = LIB + f".{os.getpid()}.tmp"
        cmd = nvcc_command(tmp, extra=("-Xptxas", "-v") if verbose else ())
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed building librps.so")
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
