"""rps_step_static: the entry point for callers that cannot allocate device memory.

A library user embedded in someone else's memory pool (or in a loop that must not
call into the driver's allocator) owns its replica and target buffers but cannot
ask for scratch.  This test drives the allocation-free entry point through the
C ABI on buffers it owns and checks that two consecutive steps give, bit for bit,
the replicas of the ordinary handle-based path (and the oracle's within the step's
tolerance), with the device's free memory unchanged across the calls.  It lives in its own file, collected
last, so a failure here cannot hide the results of the other tests.
"""
import gc
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_1810_07766_b200 import workloads as wl

pytestmark = pytest.mark.gpu

STEP_TOL = 1e-6


@pytest.mark.parametrize("name,d,n", [("cfg2", 100_010, None), ("cfg4", 50_001, None), ("cfg5", 32_768, None),
                                      # worker counts between two powers of two: the streamed kernel, both types
                                      ("cfg5", 40_008, 24), ("cfg4", 60_004, 12), ("cfg5", 30_001, 5)])
def test_static_step_matches_the_bound_step_twice_in_a_row(name, d, n, oracle):
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    from paper_1810_07766_b200 import binding, build

    build.build()
    w = wl.WORKLOADS[name].scaled(d=d, steps=2)
    if n is not None:
        w = replace(w, n=n)
    b = wl.make_targets(w)

    # the existing path: a handle with caller-lent scratch
    ref = binding.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype=w.dtype, sigma=w.sigma)
    ref.set_targets(b)
    expected = []
    for _ in range(2):
        ref.step()
        expected.append(ref.read())
    pitch = ref.pitch
    # and the oracle, from the same inputs
    oracle_x = wl.make_initial(w)
    oracle_states = []
    for t in range(2):
        oracle.step(oracle_x, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=t)
        oracle_states.append(oracle_x.copy())

    # the allocation-free path: buffers made up front, nothing allocated around the calls
    tdtype = torch.float32 if w.dtype == "f32" else torch.bfloat16
    x_dev = torch.zeros((w.n, pitch), dtype=tdtype, device="cuda")
    b_dev = ref.b_dev.clone()
    scratch_x = x_dev.clone()
    # One call on a copy first: what a first call on a device does once (it looks up the built-in array's address,
    # the kernels' code is loaded, their shared-memory attribute is set) is behind us when the memory is counted.
    binding.step_static(scratch_x, b_dev, n=w.n, d=w.d, dtype=w.dtype, p=w.p, gamma=w.gamma, sigma=w.sigma,
                        seed=w.seed, t=0)
    # tensors of earlier tests may still be waiting for the garbage collector: let them go first, so that
    # the only thing that could change the counts below is the call under test
    gc.collect()
    torch.cuda.synchronize()
    held_by_torch = torch.cuda.memory_allocated()
    free_on_device, _ = torch.cuda.mem_get_info()  # the driver's own count: sees an allocation made inside the library too
    for t in range(2):
        binding.step_static(x_dev, b_dev, n=w.n, d=w.d, dtype=w.dtype, p=w.p, gamma=w.gamma, sigma=w.sigma,
                            seed=w.seed, t=t)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] >= free_on_device   # nothing was allocated on the device, by anybody
        assert torch.cuda.memory_allocated() <= held_by_torch
        got = x_dev[:, :w.d].contiguous()
        got = (got.view(torch.int16) if w.dtype == "bf16" else got).cpu().numpy()
        if w.dtype == "bf16":
            got = got.view(np.uint16)
        # the same kernels ran on the same inputs: not one bit differs from the handle's step
        assert np.array_equal(got.view(np.uint8), expected[t].view(np.uint8))
        g, o = wl.as_float64(w, got), wl.as_float64(w, oracle_states[t])
        tol = 1e-2 if w.dtype == "bf16" else (t + 1) * STEP_TOL
        assert (np.abs(g - o) <= tol * (1 + np.abs(o))).all()
    assert not x_dev[:, w.d:].any()
    ref.close()


def test_static_step_rejects_what_it_cannot_hold():
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    from paper_1810_07766_b200 import binding, build

    build.build()
    lib = binding.load_library()
    x = torch.zeros((65, 32), dtype=torch.float32, device="cuda")
    args = (x.data_ptr(), x.data_ptr(), 32, 0.1, 0.1, 0.0, 1, 0, None)
    assert lib.rps_step_static(65, 32, 0, *args) == binding.RPS_ELIMIT      # more workers than the record holds
    assert lib.rps_step_static(0, 32, 0, *args) == binding.RPS_EINVAL
    assert lib.rps_step_static(4, 32, 0, x.data_ptr(), x.data_ptr(), 31, 0.1, 0.1, 0.0, 1, 0, None) == binding.RPS_EINVAL
    assert lib.rps_step_static(4, 32, 0, None, x.data_ptr(), 32, 0.1, 0.1, 0.0, 1, 0, None) == binding.RPS_EINVAL
    with pytest.raises(binding.RPSError):
        binding.step_static(x, x, n=65, d=32, dtype="f32", p=0.1, gamma=0.1, sigma=0.0, seed=1, t=0)
