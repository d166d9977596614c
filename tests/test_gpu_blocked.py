"""Temporal blocking of rps_step_n (rps_options.block_steps): several consecutive steps applied to a slice of x
while it sits in registers must give, bit for bit, what the same number of single steps gives in the same lane
shape, and stay within the step's tolerance of the oracle's run."""
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


def bits_of(a, dtype):
    return a.view(np.uint16 if dtype == "bf16" else np.uint32)


SHAPES = [(1, 50_001, "f32"), (2, 50_002, "f32"), (3, 40_003, "f32"), (8, 100_010, "f32"), (16, 40_009, "f32"),
          (33, 20_003, "f32"), (64, 10_007, "f32"), (3, 40_003, "bf16"), (8, 100_010, "bf16"), (32, 30_000, "bf16"),
          (64, 16_384, "bf16")]


@pytest.mark.parametrize("n,d,dtype", SHAPES)
def test_blocked_steps_equal_single_steps_bit_for_bit(rps_mod, n, d, dtype):
    w = wl.Workload("blocked", n=n, d=d, dtype=dtype, p=0.15, gamma=0.1, sigma=0.1, seed=90 + n, steps=23, hetero=True)
    b = wl.make_targets(w)
    for t0 in (0, (1 << 32) - 7):
        single = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, kernel=1, workers_per_lane=4,
                             mask_window=8)
        single.set_targets(b)
        single.set_step(t0)
        single.step_n(w.steps)
        want = single.read()
        single.close()
        for block_steps, window in ((5, 8), (8, 8), (2, 3), (23, 32)):
            r = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, mask_window=window,
                            block_steps=block_steps)
            r.set_targets(b)
            r.set_step(t0)
            r.step_n(w.steps)
            assert r.get_step() == t0 + w.steps
            if block_steps >= 5:
                # far fewer launches (mask generator included) than steps: the steps really were fused
                assert r.launch_count() <= w.steps // 2
            assert (bits_of(r.read(), dtype) == bits_of(want, dtype)).all(), (t0, block_steps, window)
            r.close()


@pytest.mark.parametrize("name", ["cfg1", "cfg4", "cfg5"])
def test_blocked_run_matches_the_oracle(rps_mod, oracle, name):
    base = {"cfg1": wl.WORKLOADS["cfg1"].scaled(d=65_536, steps=40), "cfg4": wl.WORKLOADS["cfg4"].scaled(d=100_005, steps=25),
            "cfg5": wl.WORKLOADS["cfg5"].scaled(d=65_536, steps=20)}[name]
    w = base
    b = wl.make_targets(w)
    want = wl.make_initial(w)
    oracle.run(want, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype=w.dtype, sigma=w.sigma, block_steps=16)
    r.set_targets(b)
    r.step_n(w.steps)
    got = r.read()
    r.close()
    g, o = wl.as_float64(w, got), wl.as_float64(w, want)
    tol = 1e-2 if w.dtype == "bf16" else 1e-5
    assert (np.abs(g - o) / (1.0 + np.abs(o))).max() <= tol
    assert np.linalg.norm(g - o) / np.linalg.norm(o) <= tol


def test_tracked_steps_and_gradient_averaging_stay_single(rps_mod):
    """Blocking applies to untracked model averaging only: anything else runs step by step, with the same results."""
    w = wl.Workload("mixed", n=8, d=60_010, dtype="f32", p=0.1, gamma=0.05, sigma=0.1, seed=3, steps=12)
    b = wl.make_targets(w)
    plain = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, sigma=w.sigma, kernel=1, workers_per_lane=4)
    plain.set_targets(b)
    plain.track(5)
    plain.step_n(w.steps)
    want, want_trace = plain.read(), plain.read_trace()
    plain.close()
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, sigma=w.sigma, kernel=1, workers_per_lane=4, block_steps=4)
    r.set_targets(b)
    r.track(5)            # the first five steps are tracked, hence single; the other seven are blocked
    r.step_n(w.steps)
    assert (r.read().view(np.uint32) == want.view(np.uint32)).all()
    assert np.allclose(r.read_trace(), want_trace, rtol=1e-9)
    assert 5 < r.launch_count() < w.steps + 1
    r.close()
    for average_gradients in (True,):
        a = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, sigma=w.sigma, average_gradients=average_gradients)
        c = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, sigma=w.sigma, average_gradients=average_gradients, block_steps=8)
        for h in (a, c):
            h.set_targets(b)
            h.step_n(6)
        assert (a.read().view(np.uint32) == c.read().view(np.uint32)).all()
        a.close()
        c.close()


def test_blocked_shards_reproduce_the_whole_model(rps_mod):
    w = wl.Workload("bs", n=16, d=90_011, dtype="f32", p=0.2, gamma=0.1, sigma=0.05, seed=8, steps=9)
    b = wl.make_targets(w)
    whole = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, sigma=w.sigma, block_steps=4)
    whole.set_targets(b)
    whole.step_n(w.steps)
    want = whole.read()
    whole.close()
    parts = []
    for rank in range(3):
        begin, cols = rps_mod.shard_columns(w.d, 3, rank)
        r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, sigma=w.sigma, block_steps=4, shard_begin=begin, shard_cols=cols)
        r.set_targets(np.ascontiguousarray(b[:, begin:begin + cols]))
        r.step_n(w.steps)
        parts.append(r.read())
        r.close()
    assert (np.concatenate(parts, axis=1).view(np.uint32) == want.view(np.uint32)).all()
