"""Builds ``csrc/librps.so`` in-tree with nvcc for sm_100a (no GPU needed to compile)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(CSRC, "librps.so")
SOURCES = ["rps_api.cu", "rps_kernels.cu", "rps_direct_track.cu", "rps_blocked.cu", "rps_staged.cu",
           "rps_staged_grad.cu", "rps_staged_track.cu", "rps_ring.cu", "rps_stream.cu", "rps_static.cu"]
HEADERS = ["rps_device.cuh", "rps_kernels.h", "rps_direct.cuh", "rps_staged.cuh", "rps_tma.cuh"]


def nvcc_flags(extra=()):
    return ["-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
            "-Xcompiler", "-fPIC,-Wall", "-I", INCLUDE, "-I", CSRC, *extra]


def _nvcc() -> str:
    return os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(INCLUDE, "rps.h")]
    return any(os.path.getmtime(f) > built for f in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles every .cu to an object (in parallel) and links librps.so; a no-op when up to date."""
    if not (force or is_stale()):
        return LIB
    from concurrent.futures import ThreadPoolExecutor

    obj_dir = os.path.join(CSRC, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    tag = str(os.getpid())
    extra = ("-Xptxas", "-v") if verbose else ()

    def compile_one(src):
        obj = os.path.join(obj_dir, f"{src}.{tag}.o")
        res = subprocess.run([_nvcc(), *nvcc_flags(extra), "-c", os.path.join(CSRC, src), "-o", obj],
                             capture_output=True, text=True)
        return src, obj, res

    with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
        results = list(pool.map(compile_one, SOURCES))
    failed = False
    for src, _, res in results:
        if verbose or res.returncode != 0:
            sys.stderr.write(f"==== {src}\n{res.stdout}{res.stderr}")
        failed |= res.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed building librps.so")
    tmp = LIB + f".{tag}.tmp"
    res = subprocess.run([_nvcc(), "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                          "-o", tmp, *[obj for _, obj, _ in results]], capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed linking librps.so")
    os.replace(tmp, LIB)
    for _, obj, _ in results:
        os.remove(obj)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
