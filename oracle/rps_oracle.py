"""ctypes front end of ``rps_oracle.c`` (TEST INFRASTRUCTURE ONLY).

Argument marshalling only; every number is computed by the C file next to this
one, which restates Algorithm 1 of the paper in double precision.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rps_oracle.c")
_LIB = os.path.join(_HERE, "librps_oracle.so")

ASSIGN_FIXED = 0
ASSIGN_PERM = 1
_DTYPE = {"f32": 0, "bf16": 1}

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (a second or so) when it is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    u32p = ctypes.POINTER(ctypes.c_uint32)
    u64p = ctypes.POINTER(ctypes.c_uint64)
    i32p = ctypes.POINTER(ctypes.c_int32)
    i64p = ctypes.POINTER(ctypes.c_int64)
    f64p = ctypes.POINTER(ctypes.c_double)
    vp = ctypes.c_void_p
    lib.rps_oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
    lib.rps_oracle_philox4x32_10.restype = None
    lib.rps_oracle_philox4x32.argtypes = [u32p, u32p, ctypes.c_int, u32p]
    lib.rps_oracle_philox4x32.restype = None
    lib.rps_oracle_masks.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_uint64, ctypes.c_uint64,
                                     ctypes.c_int, ctypes.c_int, u64p, u64p, i32p, i32p]
    lib.rps_oracle_masks.restype = ctypes.c_int
    lib.rps_oracle_noise.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int, ctypes.c_int64]
    lib.rps_oracle_noise.restype = ctypes.c_double
    lib.rps_oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
    lib.rps_oracle_bf16_to_double.restype = ctypes.c_double
    lib.rps_oracle_double_to_bf16.argtypes = [ctypes.c_double]
    lib.rps_oracle_double_to_bf16.restype = ctypes.c_uint16
    lib.rps_oracle_block_size.argtypes = [ctypes.c_int, ctypes.c_int64]
    lib.rps_oracle_block_size.restype = ctypes.c_int64
    lib.rps_oracle_step.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int, vp, vp, ctypes.c_double,
                                    ctypes.c_double, ctypes.c_double, ctypes.c_uint64, ctypes.c_uint64,
                                    ctypes.c_int, ctypes.c_int, u64p, u64p]
    lib.rps_oracle_step.restype = ctypes.c_int
    lib.rps_oracle_run.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int, vp, vp, ctypes.c_double,
                                   ctypes.c_double, ctypes.c_double, ctypes.c_uint64, ctypes.c_uint64,
                                   ctypes.c_int64, ctypes.c_int, ctypes.c_int]
    lib.rps_oracle_run.restype = ctypes.c_int
    lib.rps_oracle_step_gradavg.argtypes = lib.rps_oracle_step.argtypes
    lib.rps_oracle_step_gradavg.restype = ctypes.c_int
    lib.rps_oracle_run_gradavg.argtypes = lib.rps_oracle_run.argtypes
    lib.rps_oracle_run_gradavg.restype = ctypes.c_int
    lib.rps_oracle_step_columns.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int, ctypes.c_int64, i64p,
                                            vp, vp, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                            ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int, ctypes.c_int]
    lib.rps_oracle_step_columns.restype = ctypes.c_int
    lib.rps_oracle_diag.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int, vp, vp, f64p, f64p]
    lib.rps_oracle_diag.restype = ctypes.c_int
    lib.rps_oracle_alpha_mc.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_uint64, ctypes.c_uint64,
                                        ctypes.c_int64, ctypes.c_int, ctypes.c_int, f64p, f64p]
    lib.rps_oracle_alpha_mc.restype = ctypes.c_int
    _lib = lib
    return lib


def _check_state(x: np.ndarray, b: np.ndarray, dtype: str) -> Tuple[int, int]:
    want = np.float32 if dtype == "f32" else np.uint16
    for name, a in (("x", x), ("b", b)):
        if a.dtype != want or a.ndim != 2 or not a.flags.c_contiguous:
            raise ValueError(f"{name} must be a C-contiguous [n][d] array of {want.__name__}")
    if x.shape != b.shape:
        raise ValueError("x and b differ in shape")
    return x.shape


def philox4x32_10(ctr, key) -> Tuple[int, int, int, int]:
    c = (ctypes.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    out = (ctypes.c_uint32 * 4)()
    _load().rps_oracle_philox4x32_10(c, k, out)
    return tuple(int(v) for v in out)


def philox4x32(ctr, key, rounds: int) -> Tuple[int, int, int, int]:
    c = (ctypes.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    out = (ctypes.c_uint32 * 4)()
    _load().rps_oracle_philox4x32(c, k, rounds, out)
    return tuple(int(v) for v in out)


def masks(n: int, p: float, seed: int, t: int, self_delivery: bool = True, assign: int = ASSIGN_FIXED):
    """(up[n], down[n], cnt[n], server[n]) of step ``t`` as numpy arrays."""
    up = np.zeros(n, dtype=np.uint64)
    down = np.zeros(n, dtype=np.uint64)
    cnt = np.zeros(n, dtype=np.int32)
    server = np.zeros(n, dtype=np.int32)
    rc = _load().rps_oracle_masks(
        n, p, seed, t, int(self_delivery), assign,
        up.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)),
        down.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)),
        cnt.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
        server.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    if rc != 0:
        raise ValueError("rps_oracle_masks rejected its arguments")
    return up, down, cnt, server


def noise(seed: int, t: int, i: int, c: int) -> float:
    return float(_load().rps_oracle_noise(seed, t, i, c))


def bf16_to_double(bits: int) -> float:
    return float(_load().rps_oracle_bf16_to_double(bits))


def double_to_bf16(v: float) -> int:
    return int(_load().rps_oracle_double_to_bf16(v))


def block_size(n: int, d: int) -> int:
    return int(_load().rps_oracle_block_size(n, d))


def step(x: np.ndarray, b: np.ndarray, *, dtype: str, gamma: float, sigma: float, p: float, seed: int, t: int,
         self_delivery: bool = True, assign: int = ASSIGN_FIXED,
         forced_up: Optional[np.ndarray] = None, forced_down: Optional[np.ndarray] = None,
         average_gradients: bool = False) -> None:
    """One iteration of Algorithm 1 (or of its gradient-averaging comparison), in place on ``x``."""
    n, d = _check_state(x, b, dtype)
    u64p = ctypes.POINTER(ctypes.c_uint64)
    fu = fd = None
    if (forced_up is None) != (forced_down is None):
        raise ValueError("give both forced masks or neither")
    if forced_up is not None:
        fu_a = np.ascontiguousarray(forced_up, dtype=np.uint64)
        fd_a = np.ascontiguousarray(forced_down, dtype=np.uint64)
        if fu_a.shape != (n,) or fd_a.shape != (n,):
            raise ValueError("forced masks must have n entries")
        fu, fd = fu_a.ctypes.data_as(u64p), fd_a.ctypes.data_as(u64p)
    fn = _load().rps_oracle_step_gradavg if average_gradients else _load().rps_oracle_step
    rc = fn(n, d, _DTYPE[dtype], x.ctypes.data, b.ctypes.data, gamma, sigma, p, seed, t, int(self_delivery), assign,
            fu, fd)
    if rc != 0:
        raise ValueError("rps_oracle_step rejected its arguments")


def run(x: np.ndarray, b: np.ndarray, *, dtype: str, gamma: float, sigma: float, p: float, seed: int,
        t0: int, steps: int, self_delivery: bool = True, assign: int = ASSIGN_FIXED,
        average_gradients: bool = False) -> None:
    """``steps`` iterations of Algorithm 1 starting at step ``t0``, in place on ``x``."""
    n, d = _check_state(x, b, dtype)
    fn = _load().rps_oracle_run_gradavg if average_gradients else _load().rps_oracle_run
    rc = fn(n, d, _DTYPE[dtype], x.ctypes.data, b.ctypes.data, gamma, sigma, p, seed, t0, steps, int(self_delivery),
            assign)
    if rc != 0:
        raise ValueError("rps_oracle_run rejected its arguments")


def step_columns(d: int, cols: np.ndarray, x_cols: np.ndarray, b_cols: np.ndarray, *, dtype: str, gamma: float,
                 sigma: float, p: float, seed: int, t: int, self_delivery: bool = True,
                 assign: int = ASSIGN_FIXED) -> None:
    """The step on gathered columns ``cols`` of a size-``d`` model, in place on ``x_cols``."""
    n, ncols = _check_state(x_cols, b_cols, dtype)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    if cols.shape != (ncols,):
        raise ValueError("cols must list one index per gathered column")
    rc = _load().rps_oracle_step_columns(n, d, _DTYPE[dtype], ncols,
                                         cols.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                                         x_cols.ctypes.data, b_cols.ctypes.data, gamma, sigma, p, seed, t,
                                         int(self_delivery), assign)
    if rc != 0:
        raise ValueError("rps_oracle_step_columns rejected its arguments")


def diag(x: np.ndarray, b: np.ndarray, *, dtype: str) -> Tuple[float, float]:
    """(||xbar - mean_i b_i||^2, sum_i ||x^(i) - xbar||^2)."""
    n, d = _check_state(x, b, dtype)
    a = ctypes.c_double()
    c = ctypes.c_double()
    _load().rps_oracle_diag(n, d, _DTYPE[dtype], x.ctypes.data, b.ctypes.data, ctypes.byref(a), ctypes.byref(c))
    return a.value, c.value


def alpha_mc(n: int, p: float, seed: int, t0: int, steps: int, self_delivery: bool = True,
             assign: int = ASSIGN_FIXED) -> Tuple[float, float]:
    """Monte-Carlo (alpha_1, alpha_2) of Eqs. (4), (5) over the n blocks of ``steps`` steps from ``t0``."""
    a1 = ctypes.c_double()
    a2 = ctypes.c_double()
    rc = _load().rps_oracle_alpha_mc(n, p, seed, t0, steps, int(self_delivery), assign, ctypes.byref(a1),
                                     ctypes.byref(a2))
    if rc != 0:
        raise ValueError("rps_oracle_alpha_mc rejected its arguments")
    return a1.value, a2.value
