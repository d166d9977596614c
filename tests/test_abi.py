"""Host-side checks of the C ABI: the built library exports every symbol that
include/rps.h declares, and the calls that need no GPU validate their arguments."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "rps.h")


@pytest.fixture(scope="module")
def lib():
    from paper_1810_07766_b200 import build, binding

    build.build()
    return binding.load_library()


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rps_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_1810_07766_b200 import binding

    names = declared_symbols()
    assert len(names) >= 20
    assert sorted(binding.SYMBOLS) == names
    for name in names:
        assert getattr(lib, name) is not None


def test_create_validates_arguments(lib):
    h = ctypes.c_void_p()
    bad = [(0, 10, 0.1, 0.1), (65, 10, 0.1, 0.1), (4, 0, 0.1, 0.1), (4, 1 << 34, 0.1, 0.1), (4, 10, -0.1, 0.1),
           (4, 10, 1.5, 0.1), (4, 10, float("nan"), 0.1), (4, 10, 0.1, float("inf"))]
    for n, d, p, g in bad:
        assert lib.rps_create(n, d, p, g, 0, ctypes.byref(h)) == -1
        assert not h.value
        assert lib.rps_last_error(None)
    assert lib.rps_create(4, 10, 0.1, 0.1, 0, None) == -1
    assert lib.rps_destroy(None) == 0


def test_options_pitch_and_state_errors(lib):
    from paper_1810_07766_b200.binding import rps_options

    h = ctypes.c_void_p()
    assert lib.rps_create(8, 11_173_962, 0.1, 0.05, 1, ctypes.byref(h)) == 0
    try:
        assert lib.rps_pitch(h) == 11_174_144                      # rounded up to a whole number of kilobytes
        opt = rps_options()
        assert lib.rps_default_options(ctypes.byref(opt)) == 0
        assert (opt.dtype, opt.assign, opt.self_delivery, opt.mask_window, opt.sigma) == (0, 0, 1, 32, 0.0)
        assert (opt.kernel, opt.workers_per_lane, opt.stages, opt.consumer_warps) == (0, 0, 0, 0)
        assert opt.row_skew_lines == -1 and opt.copy_mode == 0 and opt.slice_bytes == 0 and opt.store_mode == 0
        assert opt.wait_limit_ms == 0 and opt.withhold_copies == 0 and opt.average == 0
        assert opt.traversal == 0 and opt.l2_policy == 0 and opt.launch_overlap == 0
        assert opt.shard_begin == 0 and opt.shard_cols == 0 and opt.block_steps == 0 and opt.team_warps == 0
        assert opt.early_targets == 0 and opt.fuse_steps == 0
        assert lib.rps_scratch_bytes(h) == 256 + 34 * 1792
        opt.dtype = 1
        assert lib.rps_configure(h, ctypes.byref(opt)) == 0
        assert lib.rps_pitch(h) == 11_174_400                      # the same in bf16
        for field, value in (("dtype", 7), ("assign", 2), ("self_delivery", 3), ("mask_window", 0),
                             ("mask_window", 257), ("sigma", -1.0), ("kernel", 5), ("workers_per_lane", 3), ("stages", 1),
                             ("stages", 9), ("consumer_warps", 33), ("slice_bytes", 4), ("store_mode", 4), ("wait_limit_ms", -1), ("withhold_copies", 2), ("average", 2), ("row_skew_lines", -2), ("copy_mode", 3),
                             ("traversal", 2), ("l2_policy", 3), ("launch_overlap", 3),
                             ("shard_cols", -1), ("shard_begin", 64), ("shard_cols", 11_173_963),
                             ("block_steps", -1), ("block_steps", 33), ("team_warps", -1), ("team_warps", 17),
                             ("early_targets", -1), ("early_targets", 3), ("fuse_steps", -1), ("fuse_steps", 3)):
            bad = rps_options()
            lib.rps_default_options(ctypes.byref(bad))
            setattr(bad, field, value)
            assert lib.rps_configure(h, ctypes.byref(bad)) == -1
            assert lib.rps_last_error(h)
        # a shard starts at a multiple of 64 columns and ends inside the model; its pitch is its own
        shard = rps_options()
        lib.rps_default_options(ctypes.byref(shard))
        shard.shard_begin, shard.shard_cols = 100, 1000
        assert lib.rps_configure(h, ctypes.byref(shard)) == -1
        shard.shard_begin, shard.shard_cols = 11_173_952, 11
        assert lib.rps_configure(h, ctypes.byref(shard)) == -1
        shard.shard_begin, shard.shard_cols = 11_173_952, 10
        assert lib.rps_configure(h, ctypes.byref(shard)) == 0
        assert lib.rps_pitch(h) == 256                                 # a shard of 10 floats: one kilobyte per row
        shard.shard_begin, shard.shard_cols = 0, 0
        shard.dtype = 1
        assert lib.rps_configure(h, ctypes.byref(shard)) == 0
        # nothing is bound yet: stepping is a state error, not a crash
        assert lib.rps_step(h) == -2
        assert lib.rps_step_n(h, 3) == -2
        assert lib.rps_read(h, None) == -2
        assert lib.rps_track(h, None, 4) == -2
        a1, a2 = ctypes.c_double(), ctypes.c_double()
        assert lib.rps_estimate_alpha(h, 0, 10, ctypes.byref(a1), ctypes.byref(a2)) == -2
        count = ctypes.c_int64()
        assert lib.rps_read_trace(h, None, 0, ctypes.byref(count)) == -2
        assert b"rps_bind" in lib.rps_last_error(h)
        assert lib.rps_bind(h, None, None, 0, None, 0, None) == -1
        t = ctypes.c_uint64()
        assert lib.rps_set_step(h, 1 << 40) == 0 and lib.rps_get_step(h, ctypes.byref(t)) == 0
        assert t.value == 1 << 40
        assert lib.rps_launch_count(h) == 0
    finally:
        assert lib.rps_destroy(h) == 0
    assert lib.rps_version() == b"0.1"


def test_binding_refuses_to_run_without_a_gpu():
    import torch

    from paper_1810_07766_b200 import binding

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        binding.RPS(4, 16, 0.1, 0.1, 0)
