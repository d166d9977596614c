"""Distinct handles are independent: stepped from different host threads, on streams of their own, they give bit
for bit what each gives alone.  (What the launch wrappers remember about a kernel, the shared memory it has been
granted and its occupancy, is kept per device under a lock.)  A call made with another device current than the one
the handle was bound on is refused."""
import threading

import numpy as np
import pytest
import torch

from paper_1810_07766_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rps_mod():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_1810_07766_b200 import binding, build

    build.build()
    binding.load_library()
    return binding


JOBS = [
    # (n, d, dtype, options): the same instantiation twice (two seeds), and one each of the other kernels
    (8, 300_001, "f32", {}), (8, 300_001, "f32", {}), (64, 100_003, "bf16", {}), (64, 100_003, "bf16", {}),
    (16, 200_005, "bf16", {}), (32, 90_001, "f32", {}), (4, 4097, "f32", {}), (12, 70_001, "f32", dict(kernel=4)),
]


def run_job(rps_mod, k, job, steps, own_stream, out, errors):
    try:
        n, d, dtype, opts = job
        w = wl.Workload("threads", n=n, d=d, dtype=dtype, p=0.15, gamma=0.05, sigma=0.1, seed=50 + k, steps=steps)
        b = wl.make_targets(w)
        stream = torch.cuda.Stream() if own_stream else None
        r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, stream=stream, **opts)
        r.set_targets(b)
        for _ in range(steps):  # one call per step: the threads' launches interleave
            r.step()
        out[k] = r.read()
        r.close()
    except Exception as exc:  # reported by the test's thread
        errors.append((k, repr(exc)))


def test_handles_stepped_from_several_threads_equal_the_same_handles_alone(rps_mod):
    steps = 12
    alone, together, errors = {}, {}, []
    for k, job in enumerate(JOBS):
        run_job(rps_mod, k, job, steps, False, alone, errors)
    assert not errors, errors
    for _ in range(3):
        threads = [threading.Thread(target=run_job, args=(rps_mod, k, job, steps, True, together, errors))
                   for k, job in enumerate(JOBS)]
        for t in threads:
            t.start()
        for t in threads:
            t.join()
        assert not errors, errors
        for k in range(len(JOBS)):
            assert np.array_equal(alone[k].view(np.uint8), together[k].view(np.uint8)), JOBS[k]


def test_a_call_with_another_device_current_is_refused(rps_mod):
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two visible devices")
    r = rps_mod.RPS(4, 1000, 0.1, 0.1, 1, device="cuda:0")
    with torch.cuda.device(1):
        # the binding makes the handle's device current; the library itself refuses
        rc = r._lib.rps_step(r._h)
        assert rc == rps_mod.RPS_ESTATE
        r.step()  # through the binding: fine
    r.close()
    # a second device runs the same instantiations with its own granted shared memory
    w = wl.Workload("threads", n=8, d=300_001, dtype="f32", p=0.15, gamma=0.05, sigma=0.1, seed=3, steps=3)
    b = wl.make_targets(w)
    got = []
    for dev in ("cuda:0", "cuda:1"):
        r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, sigma=w.sigma, device=dev)
        r.set_targets(b)
        r.step_n(3)
        got.append(r.read())
        r.close()
    assert np.array_equal(got[0], got[1])
