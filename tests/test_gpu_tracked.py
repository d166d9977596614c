"""Tracked steps (rps_track): the distance to the optimum and the consensus error that the fused
pass reports as a by-product must equal the oracle's diagnostics of the state that same step left
in memory, and tracking must not change that state.

Expected values come from the oracle alone: its diag() of the replicas read back after every step,
and its own free run from the same seeded inputs.
"""
import numpy as np
import pytest
import torch

from paper_1810_07766_b200 import workloads as wl

pytestmark = pytest.mark.gpu

# fp32 sums relative to a per-column pivot, fp64 across tiles: see the derivation next to the tolerance
# of the step itself; the observed error is ~1e-6
TRACE_RTOL = 1e-4


@pytest.fixture(scope="module")
def rps_mod():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_1810_07766_b200 import binding, build

    build.build()
    binding.load_library()
    return binding


def close(got, want, scale):
    return abs(got - want) <= TRACE_RTOL * abs(want) + 1e-12 * scale


SHAPES = [
    # n, d, dtype: every lane-group count of the 4-workers-per-lane family, ragged rows and blocks, workers
    # that do not fill the last lane group (3, 6, 33)
    (1, 70_001, "f32"), (2, 70_002, "f32"), (3, 70_003, "f32"), (4, 65_536, "f32"), (6, 50_001, "f32"),
    (8, 100_010, "f32"), (16, 40_009, "f32"), (32, 20_005, "f32"), (33, 20_003, "f32"), (64, 10_007, "f32"),
    (1, 70_001, "bf16"), (3, 70_003, "bf16"), (8, 100_010, "bf16"), (16, 40_009, "bf16"), (33, 20_003, "bf16"),
    (64, 16_384, "bf16"),
]


@pytest.mark.parametrize("n,d,dtype", SHAPES)
@pytest.mark.parametrize("average_gradients", [False, True])
def test_trace_equals_the_oracle_diagnostics_of_the_state_left_behind(rps_mod, oracle, n, d, dtype, average_gradients):
    w = wl.Workload("tracked", n=n, d=d, dtype=dtype, p=0.2, gamma=0.1, sigma=0.1, seed=77 + n, steps=4,
                    hetero=True)
    b = wl.make_targets(w)
    worst = 0.0
    for kernel, store_mode, copy_mode in ((1, 0, 0), (2, 1, 1), (2, 2, 2), (2, 3, 0), (4, 0, 0)):
        r = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, kernel=kernel, store_mode=store_mode,
                        copy_mode=copy_mode, average_gradients=average_gradients)
        r.set_targets(b)
        r.track(w.steps)
        states = []
        for _ in range(w.steps):
            r.step()
            states.append(r.read())
        trace = r.read_trace()
        assert trace.shape == (w.steps, 2)
        for k, x in enumerate(states):
            dist2, cons = oracle.diag(x, b, dtype=dtype)
            assert close(trace[k, 0], dist2, n * d), (kernel, store_mode, k, trace[k, 0], dist2)
            assert close(trace[k, 1], cons, n * d), (kernel, store_mode, k, trace[k, 1], cons)
            worst = max(worst, abs(trace[k, 0] - dist2) / max(dist2, 1e-300),
                        abs(trace[k, 1] - cons) / max(cons, 1e-300) if cons > 0 else 0.0)
        # the device's own off-path reduction agrees too
        dist2, cons = r.diag()
        assert close(trace[-1, 0], dist2, n * d) and close(trace[-1, 1], cons, n * d)
        r.close()
    if n == 1:
        assert (trace[:, 1] == 0.0).all()  # one worker: no consensus error at all


@pytest.mark.parametrize("name", ["cfg1", "cfg3", "cfg5"])
def test_trace_follows_the_oracle_run(rps_mod, oracle, name):
    """Free-running: the trace against the oracle's diagnostics of its own run (never the GPU's state)."""
    base = {"cfg1": wl.WORKLOADS["cfg1"], "cfg3": wl.WORKLOADS["cfg3"].scaled(d=100_008, steps=40),
            "cfg5": wl.WORKLOADS["cfg5"].scaled(d=65_536, steps=20)}[name]
    w = base.scaled(d=base.d, steps=min(base.steps, 30))
    b = wl.make_targets(w)
    x = wl.make_initial(w)
    want = []
    for t in range(w.steps):
        oracle.step(x, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=t)
        want.append(oracle.diag(x, b, dtype=w.dtype))
    want = np.array(want)
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype=w.dtype, sigma=w.sigma)
    r.set_targets(b)
    r.track(w.steps)
    r.step_n(w.steps)
    trace = r.read_trace()
    r.close()
    # the states differ by the step's own tolerance (1e-5 relative for fp32, 1e-2 for bf16 replicas, whose
    # rounding decisions may differ), and so do their diagnostics
    rtol = 5e-2 if w.dtype == "bf16" else 1e-3
    assert np.allclose(trace, want, rtol=rtol, atol=0.0), np.abs(trace / want - 1.0).max()
    # the averaged model closes in on the optimum by about (1 - gamma) per step
    shrink = (1.0 - w.gamma) ** (2 * (w.steps - 1))
    assert trace[-1, 0] < max(2.0 * shrink, 0.05) * trace[0, 0]


def test_tracking_does_not_change_the_step(rps_mod):
    """Same lane shape with and without tracking: bit-identical replicas (the by-product only reads registers)."""
    for dtype, n, d in (("f32", 8, 100_010), ("bf16", 16, 65_544), ("f32", 33, 20_003)):
        w = wl.Workload("same", n=n, d=d, dtype=dtype, p=0.1, gamma=0.05, sigma=0.1, seed=5, steps=5)
        b = wl.make_targets(w)
        out = []
        for tracked in (False, True):
            for kernel in (1, 2):
                r = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, kernel=kernel,
                                workers_per_lane=4)
                r.set_targets(b)
                if tracked:
                    r.track(w.steps)
                r.step_n(w.steps)
                out.append(r.read().view(np.uint16 if dtype == "bf16" else np.uint32))
                r.close()
        for other in out[1:]:
            assert (other == out[0]).all()


def test_capacity_and_switching_off(rps_mod, oracle):
    w = wl.Workload("cap", n=4, d=50_000, dtype="f32", p=0.1, gamma=0.1, sigma=0.0, seed=3, steps=6)
    b = wl.make_targets(w)
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype="f32")
    r.set_targets(b)
    with pytest.raises(rps_mod.RPSError):
        r.read_trace()
    r.track(3)
    assert r.read_trace().shape == (0, 2)
    r.step_n(2)
    assert r.read_trace().shape == (2, 2)
    r.step_n(4)  # the last three run untracked
    trace = r.read_trace()
    assert trace.shape == (3, 2)
    # a second round of tracking starts from a cleared array and from the current state
    r.track(2)
    r.step()
    dist2, cons = oracle.diag(r.read(), b, dtype="f32")
    again = r.read_trace()
    assert again.shape == (1, 2) and close(again[0, 0], dist2, w.n * w.d) and close(again[0, 1], cons, w.n * w.d)
    r.track(0)
    with pytest.raises(rps_mod.RPSError):
        r.read_trace()
    r.step()
    r.close()
