"""ctypes binding of ``librps.so`` (the C ABI declared in ``include/rps.h``).

Argument marshalling only: every step of the method runs in the CUDA kernels of
the library.  PyTorch supplies device memory and the stream, nothing else.
There is no CPU fallback: a missing library or a failing call raises.
"""
from __future__ import annotations

import ctypes
import functools
import os
from typing import Optional, Tuple

import numpy as np
import torch

_CSRC = os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc")
LIB_PATH = os.path.join(_CSRC, "librps.so")

RPS_OK, RPS_EINVAL, RPS_ESTATE, RPS_ECUDA, RPS_ENOMEM = 0, -1, -2, -3, -4
RPS_ELIMIT = -5
RPS_F32, RPS_BF16 = 0, 1
RPS_ASSIGN_FIXED, RPS_ASSIGN_PERM = 0, 1
_DTYPE = {"f32": RPS_F32, "bf16": RPS_BF16}

# every symbol include/rps.h declares
SYMBOLS = (
    "rps_create", "rps_destroy", "rps_default_options", "rps_configure", "rps_pitch", "rps_scratch_bytes",
    "rps_bind", "rps_set_targets", "rps_write", "rps_set_step", "rps_get_step", "rps_step", "rps_step_n",
    "rps_step_forced", "rps_step_host", "rps_read", "rps_read_masks", "rps_diag", "rps_estimate_alpha", "rps_track",
    "rps_read_trace",
    "rps_profile",
    "rps_profile_read", "rps_launch_count", "rps_last_error", "rps_version", "rps_step_static",
)


class rps_options(ctypes.Structure):
    _fields_ = [("dtype", ctypes.c_int32), ("assign", ctypes.c_int32), ("self_delivery", ctypes.c_int32),
                ("mask_window", ctypes.c_int32), ("sigma", ctypes.c_double), ("row_skew_lines", ctypes.c_int32),
                ("kernel", ctypes.c_int32),
                ("workers_per_lane", ctypes.c_int32), ("stages", ctypes.c_int32), ("consumer_warps", ctypes.c_int32),
                ("copy_mode", ctypes.c_int32), ("slice_bytes", ctypes.c_int32),
                ("store_mode", ctypes.c_int32), ("wait_limit_ms", ctypes.c_int32),
                ("withhold_copies", ctypes.c_int32), ("average", ctypes.c_int32),
                ("traversal", ctypes.c_int32), ("l2_policy", ctypes.c_int32), ("launch_overlap", ctypes.c_int32),
                ("shard_begin", ctypes.c_int64), ("shard_cols", ctypes.c_int64), ("block_steps", ctypes.c_int32),
                ("team_warps", ctypes.c_int32), ("early_targets", ctypes.c_int32), ("fuse_steps", ctypes.c_int32)]


def shard_columns(d: int, world: int, rank: int, align: int = 64) -> Tuple[int, int]:
    """(shard_begin, shard_cols) of rank ``rank`` when a model of ``d`` columns is cut over ``world`` handles:
    contiguous ranges that cover [0, d) once, each starting at a multiple of ``align`` columns, sizes within one
    unit of ``align`` of each other (ranks past the end of a very short model get no columns: (d, 0))."""
    if not (0 <= rank < world) or d < 1 or align < 1:
        raise ValueError("need 0 <= rank < world, d >= 1, align >= 1")
    units = -(-d // align)                      # whole or partial units of `align` columns
    first = (units * rank) // world
    last = (units * (rank + 1)) // world
    begin, end = min(first * align, d), min(last * align, d)
    return begin, end - begin


def _device_current(method):
    """Runs a method of RPS with the handle's device current: the library launches on the current device and
    refuses a call made with another one current (RPS_ESTATE)."""
    @functools.wraps(method)
    def wrapper(self, *args, **kwargs):
        if torch.cuda.current_device() == self.device.index:
            return method(self, *args, **kwargs)
        with torch.cuda.device(self.device):
            return method(self, *args, **kwargs)
    return wrapper


class RPSError(RuntimeError):
    def __init__(self, code: int, where: str, why: str):
        super().__init__(f"{where} failed with status {code}: {why}")
        self.code = code


_lib = None


def load_library(path: str = LIB_PATH) -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} is missing: build it with `python -m paper_1810_07766_b200.build` (needs nvcc)")
    lib = ctypes.CDLL(path)
    vp, i64, u64, dbl, cint = ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64, ctypes.c_double, ctypes.c_int
    u64p, i32p, i64p, dblp = (ctypes.POINTER(t) for t in (u64, ctypes.c_int32, i64, dbl))
    sig = {
        "rps_create": (cint, [cint, i64, dbl, dbl, u64, ctypes.POINTER(vp)]),
        "rps_destroy": (cint, [vp]),
        "rps_default_options": (cint, [ctypes.POINTER(rps_options)]),
        "rps_configure": (cint, [vp, ctypes.POINTER(rps_options)]),
        "rps_pitch": (i64, [vp]),
        "rps_scratch_bytes": (ctypes.c_size_t, [vp]),
        "rps_bind": (cint, [vp, vp, vp, i64, vp, ctypes.c_size_t, vp]),
        "rps_set_targets": (cint, [vp, vp]),
        "rps_write": (cint, [vp, vp]),
        "rps_set_step": (cint, [vp, u64]),
        "rps_get_step": (cint, [vp, u64p]),
        "rps_step": (cint, [vp]),
        "rps_step_n": (cint, [vp, i64]),
        "rps_step_forced": (cint, [vp, u64p, u64p]),
        "rps_step_host": (cint, [vp, vp, vp]),
        "rps_read": (cint, [vp, vp]),
        "rps_read_masks": (cint, [vp, u64, u64p, u64p, i32p, i32p]),
        "rps_diag": (cint, [vp, dblp, dblp]),
        "rps_estimate_alpha": (cint, [vp, u64, i64, dblp, dblp]),
        "rps_track": (cint, [vp, vp, i64]),
        "rps_read_trace": (cint, [vp, vp, i64, i64p]),
        "rps_profile": (cint, [vp, cint]),
        "rps_profile_read": (cint, [vp, dblp, i64p, dblp, i64p]),
        "rps_launch_count": (i64, [vp]),
        "rps_last_error": (ctypes.c_char_p, [vp]),
        "rps_version": (ctypes.c_char_p, []),
        "rps_step_static": (cint, [cint, i64, cint, vp, vp, i64, dbl, dbl, dbl, u64, u64, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _host_ptr(a) -> int:
    """Address of a dense host array given as numpy array or CPU torch tensor."""
    if isinstance(a, torch.Tensor):
        if a.is_cuda or not a.is_contiguous():
            raise ValueError("expected a contiguous CPU tensor")
        return a.data_ptr()
    if not a.flags.c_contiguous:
        raise ValueError("expected a C-contiguous array")
    return a.ctypes.data


class RPS:
    """One simulated cluster of ``n`` workers and ``n`` parameter servers on the current GPU.

    Method names follow the C ABI (``rps_step`` -> ``step`` and so on).
    """

    def __init__(self, n: int, d: int, p: float, gamma: float, seed: int, *, dtype: str = "f32", sigma: float = 0.0,
                 assign: int = RPS_ASSIGN_FIXED, self_delivery: bool = True, mask_window: int = 32,
                 average_gradients: bool = False, shard_begin: int = 0, shard_cols: int = 0, block_steps: int = 0,
                 kernel: int = 0, workers_per_lane: int = 0, stages: int = 0, consumer_warps: int = 0,
                 row_skew_lines: int = -1, copy_mode: int = 0, slice_bytes: int = 0, store_mode: int = 0,
                 early_targets: int = 0, fuse_steps: int = 0,
                 traversal: int = 0, l2_policy: int = 0, launch_overlap: int = 0, team_warps: int = 0,
                 wait_limit_ms: int = 0, withhold_copies: bool = False,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        if not torch.cuda.is_available():
            raise RuntimeError("the RPS library needs a CUDA device; there is no CPU path")
        self.n, self.d, self.dtype = int(n), int(d), dtype
        self.cols = int(shard_cols) if shard_cols else int(d)  # columns this handle holds: its shard, or the model
        rc = self._lib.rps_create(n, d, p, gamma, seed, ctypes.byref(self._h))
        if rc != RPS_OK:
            raise RPSError(rc, "rps_create", self._lib.rps_last_error(None).decode())
        opt = rps_options()
        self._lib.rps_default_options(ctypes.byref(opt))
        opt.dtype, opt.assign, opt.self_delivery = _DTYPE[dtype], assign, int(self_delivery)
        opt.mask_window, opt.sigma = mask_window, sigma
        opt.kernel, opt.workers_per_lane, opt.stages = kernel, workers_per_lane, stages
        opt.consumer_warps = consumer_warps
        opt.row_skew_lines, opt.copy_mode, opt.slice_bytes = row_skew_lines, copy_mode, slice_bytes
        opt.store_mode, opt.wait_limit_ms, opt.withhold_copies = store_mode, wait_limit_ms, int(withhold_copies)
        opt.average = int(average_gradients)
        opt.traversal, opt.l2_policy, opt.launch_overlap = traversal, l2_policy, launch_overlap
        opt.shard_begin, opt.shard_cols, opt.block_steps = shard_begin, shard_cols, block_steps
        opt.team_warps = team_warps
        opt.early_targets = early_targets
        opt.fuse_steps = fuse_steps
        self._check(self._lib.rps_configure(self._h, ctypes.byref(opt)), "rps_configure")
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.pitch = int(self._lib.rps_pitch(self._h))
        tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
        with torch.cuda.device(self.device):
            # device memory comes from torch; the library only borrows it
            self.x_dev = torch.zeros((n, self.pitch), dtype=tdtype, device=self.device)
            self.b_dev = torch.zeros((n, self.pitch), dtype=tdtype, device=self.device)
            self.scratch = torch.zeros(int(self._lib.rps_scratch_bytes(self._h)) + 256, dtype=torch.uint8,
                                       device=self.device)
            self.stream = torch.cuda.current_stream(self.device) if stream is None else stream
            scratch_ptr = (self.scratch.data_ptr() + 255) // 256 * 256
            self._check(self._lib.rps_bind(self._h, self.x_dev.data_ptr(), self.b_dev.data_ptr(), self.pitch,
                                           scratch_ptr, self.scratch.numel() - (scratch_ptr - self.scratch.data_ptr()),
                                           self.stream.cuda_stream), "rps_bind")

    # ------------------------------------------------------------------ plumbing
    def _check(self, rc: int, where: str) -> None:
        if rc != RPS_OK:
            raise RPSError(rc, where, self._lib.rps_last_error(self._h).decode())

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            torch.cuda.synchronize(self.device)
            self._lib.rps_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _host_array(self) -> np.ndarray:
        return np.empty((self.n, self.cols), dtype=np.float32 if self.dtype == "f32" else np.uint16)

    def _expect(self, a, name: str) -> None:
        want = (self.n, self.cols)
        if tuple(a.shape) != want:
            raise ValueError(f"{name} must have shape {want}")
        size = a.element_size() if isinstance(a, torch.Tensor) else a.dtype.itemsize
        if size != (4 if self.dtype == "f32" else 2):
            raise ValueError(f"{name} has the wrong element size for {self.dtype} replicas")

    # ------------------------------------------------------------------ C ABI, one method per call
    @_device_current
    def set_targets(self, b_host) -> None:
        self._expect(b_host, "b_host")
        self._check(self._lib.rps_set_targets(self._h, _host_ptr(b_host)), "rps_set_targets")

    @_device_current
    def write(self, x_host) -> None:
        self._expect(x_host, "x_host")
        self._check(self._lib.rps_write(self._h, _host_ptr(x_host)), "rps_write")

    def set_step(self, t: int) -> None:
        self._check(self._lib.rps_set_step(self._h, t), "rps_set_step")

    def get_step(self) -> int:
        t = ctypes.c_uint64()
        self._check(self._lib.rps_get_step(self._h, ctypes.byref(t)), "rps_get_step")
        return t.value

    @_device_current
    def step(self) -> None:
        self._check(self._lib.rps_step(self._h), "rps_step")

    @_device_current
    def step_n(self, steps: int) -> None:
        self._check(self._lib.rps_step_n(self._h, steps), "rps_step_n")

    @_device_current
    def step_forced(self, up, down) -> None:
        up = np.ascontiguousarray(up, dtype=np.uint64)
        down = np.ascontiguousarray(down, dtype=np.uint64)
        if up.shape != (self.n,) or down.shape != (self.n,):
            raise ValueError("masks must have n entries")
        u64p = ctypes.POINTER(ctypes.c_uint64)
        self._check(self._lib.rps_step_forced(self._h, up.ctypes.data_as(u64p), down.ctypes.data_as(u64p)),
                    "rps_step_forced")

    @_device_current
    def step_host(self, x_host, b_host=None) -> None:
        self._expect(x_host, "x_host")
        if b_host is not None:
            self._expect(b_host, "b_host")
        self._check(self._lib.rps_step_host(self._h, _host_ptr(x_host), None if b_host is None else _host_ptr(b_host)),
                    "rps_step_host")

    @_device_current
    def read(self, out=None):
        out = self._host_array() if out is None else out
        self._expect(out, "out")
        self._check(self._lib.rps_read(self._h, _host_ptr(out)), "rps_read")
        return out

    @_device_current
    def read_masks(self, t: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
        up = np.zeros(self.n, dtype=np.uint64)
        down = np.zeros(self.n, dtype=np.uint64)
        cnt = np.zeros(self.n, dtype=np.int32)
        server = np.zeros(self.n, dtype=np.int32)
        u64p, i32p = ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_int32)
        self._check(self._lib.rps_read_masks(self._h, t, up.ctypes.data_as(u64p), down.ctypes.data_as(u64p),
                                             cnt.ctypes.data_as(i32p), server.ctypes.data_as(i32p)), "rps_read_masks")
        return up, down, cnt, server

    @_device_current
    def diag(self) -> Tuple[float, float]:
        a, c = ctypes.c_double(), ctypes.c_double()
        self._check(self._lib.rps_diag(self._h, ctypes.byref(a), ctypes.byref(c)), "rps_diag")
        return a.value, c.value

    @_device_current
    def estimate_alpha(self, t0: int, steps: int) -> Tuple[float, float]:
        """Monte-Carlo (alpha_1, alpha_2) of Eqs. (4), (5) from the drop masks of ``steps`` steps from ``t0``."""
        a1, a2 = ctypes.c_double(), ctypes.c_double()
        self._check(self._lib.rps_estimate_alpha(self._h, t0, steps, ctypes.byref(a1), ctypes.byref(a2)),
                    "rps_estimate_alpha")
        return a1.value, a2.value

    @_device_current
    def track(self, capacity: int) -> None:
        """Records {dist2_to_opt, consensus} of the state each of the next `capacity` steps leaves behind, as a
        by-product of the fused pass (rps_track); 0 switches tracking off."""
        self.trace_dev = torch.zeros((capacity, 2), dtype=torch.float64, device=self.device) if capacity > 0 else None
        ptr = self.trace_dev.data_ptr() if capacity > 0 else None
        with torch.cuda.device(self.device):
            self._check(self._lib.rps_track(self._h, ptr, capacity), "rps_track")

    @_device_current
    def read_trace(self) -> np.ndarray:
        """The recorded pairs so far as a float64 array [steps][2] (synchronises)."""
        held = getattr(self, "trace_dev", None)
        out = np.zeros((held.shape[0] if held is not None else 1, 2), dtype=np.float64)
        count = ctypes.c_int64()
        with torch.cuda.device(self.device):
            self._check(self._lib.rps_read_trace(self._h, out.ctypes.data, out.shape[0], ctypes.byref(count)),
                        "rps_read_trace")
        return out[:count.value]

    @_device_current
    def profile(self, enable: bool) -> None:
        self._check(self._lib.rps_profile(self._h, int(enable)), "rps_profile")

    @_device_current
    def profile_read(self):
        """(fused_ms, fused_launches, mask_ms, mask_launches) since profiling was enabled; resets them."""
        fm, mm = ctypes.c_double(), ctypes.c_double()
        fl, ml = ctypes.c_int64(), ctypes.c_int64()
        self._check(self._lib.rps_profile_read(self._h, ctypes.byref(fm), ctypes.byref(fl), ctypes.byref(mm),
                                               ctypes.byref(ml)), "rps_profile_read")
        return fm.value, fl.value, mm.value, ml.value

    def launch_count(self) -> int:
        return int(self._lib.rps_launch_count(self._h))


def step_static(x_dev: torch.Tensor, b_dev: torch.Tensor, *, n: int, d: int, dtype: str, p: float, gamma: float,
                sigma: float, seed: int, t: int, stream: Optional[torch.cuda.Stream] = None) -> None:
    """``rps_step_static``: one step on caller-owned ``[n][pitch]`` device tensors, for callers
    that may not allocate device memory; the library uses its built-in mask record instead of
    a scratch buffer.  Advances nothing: pass ``t`` yourself."""
    if not (x_dev.is_cuda and b_dev.is_cuda and x_dev.is_contiguous() and b_dev.is_contiguous()):
        raise ValueError("x_dev and b_dev must be contiguous CUDA tensors")
    if x_dev.dim() != 2 or x_dev.shape != b_dev.shape or x_dev.shape[0] != n:
        raise ValueError("x_dev and b_dev must both be [n][pitch]")
    stream = torch.cuda.current_stream(x_dev.device) if stream is None else stream
    with torch.cuda.device(x_dev.device):
        rc = load_library().rps_step_static(n, d, _DTYPE[dtype], x_dev.data_ptr(), b_dev.data_ptr(), x_dev.shape[1],
                                            p, gamma, sigma, seed, t, stream.cuda_stream)
    if rc != RPS_OK:
        reason = {RPS_EINVAL: "bad argument", RPS_ELIMIT: "n exceeds the built-in mask record (64 workers)",
                  RPS_ECUDA: "CUDA error"}.get(rc, "error")
        raise RPSError(rc, "rps_step_static", reason)


def version() -> str:
    return load_library().rps_version().decode()
