"""The self-refilling ring (kernel 3: every warp computes, the last reader of a stage refills it) against the
oracle, and bit for bit against the staged kernel in the same lane shape: the two run the same arithmetic on the
same lanes, so not one bit of x may differ, whatever the teams, the ring depth, the traversal or the shard."""
import numpy as np
import pytest
import torch

from paper_1810_07766_b200 import workloads as wl

pytestmark = pytest.mark.gpu

BF16_TOL = 1e-2


@pytest.fixture(scope="module")
def rps_mod():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_1810_07766_b200 import binding, build

    build.build()
    binding.load_library()
    return binding


def run(rps_mod, w, b, x0, steps, t0=0, shard=None, **opts):
    begin, cols = shard if shard else (0, w.d)
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype=w.dtype, sigma=w.sigma,
                    shard_begin=begin if shard else 0, shard_cols=cols if shard else 0, **opts)
    r.set_targets(np.ascontiguousarray(b[:, begin:begin + cols]))
    r.write(np.ascontiguousarray(x0[:, begin:begin + cols]))
    r.x_dev[:, cols:] = 3.0  # sentinel in the padding between the last column and the row pitch
    r.set_step(t0)
    r.step_n(steps)
    got = r.read()
    unit = 8
    edge = -(-cols // unit) * unit
    assert (r.x_dev[:, edge:].float() == 3.0).all(), "padding was written"
    r.close()
    return got


SHAPES = [
    # n, d: every lane-group count (n <= 8, 16, 32, 64), n that leaves lanes without a worker, ragged d, one tile and many
    (5, 70_003), (8, 262_144), (9, 1031), (16, 131_075), (17, 4097), (32, 65_536), (33, 20_011), (48, 50_001),
    (63, 8191), (64, 65_536), (64, 300_007), (64, 7), (6, 1),
]


@pytest.mark.parametrize("n,d", SHAPES)
def test_ring_equals_the_staged_kernel_bit_for_bit_and_the_oracle(rps_mod, oracle, n, d):
    w = wl.Workload("ring", n=n, d=d, dtype="bf16", p=0.2, gamma=0.05, sigma=0.1, seed=900 + n, steps=5, hetero=True)
    b = wl.make_targets(w)
    x0 = wl.f32_to_bf16_bits(np.random.default_rng(n * 7 + 1).standard_normal((n, d)).astype(np.float32))
    want = x0.copy()
    oracle.run(want, b, dtype="bf16", gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=3, steps=w.steps)
    ref = run(rps_mod, w, b, x0, w.steps, t0=3, kernel=2, workers_per_lane=8, store_mode=1)
    for store_mode in (1, 2, 3):  # from registers; TMA tensor stores from an output tile; from the x tile in place
        for team_warps, stages in ((0, 0), (1, 2), (2, 0), (4, 3), (8, 2), (16, 0), (4, 8), (12, 0), (3, 5), (7, 2)):
            got = run(rps_mod, w, b, x0, w.steps, t0=3, kernel=3, team_warps=team_warps, stages=stages,
                      store_mode=store_mode)
            assert (got == ref).all(), (store_mode, team_warps, stages, int((got != ref).sum()))
    g, o = wl.as_float64(w, ref), wl.as_float64(w, want)
    assert (np.abs(g - o) / (1 + np.abs(o))).max() <= BF16_TOL


def test_ring_options_do_not_change_a_bit(rps_mod):
    """Traversal, launch overlap, the mask window and column shards leave the ring kernel's result as they leave
    the staged kernel's: the whole model in one handle, upwards, is the reference."""
    w = wl.Workload("ring", n=64, d=200_017, dtype="bf16", p=0.1, gamma=0.02, sigma=0.1, seed=77, steps=6)
    b = wl.make_targets(w)
    x0 = wl.f32_to_bf16_bits(np.random.default_rng(5).standard_normal((w.n, w.d)).astype(np.float32))
    ref = run(rps_mod, w, b, x0, w.steps, kernel=3, traversal=1)
    for store_mode in (1, 2, 3):
        for opts in (dict(traversal=0), dict(launch_overlap=1), dict(mask_window=1), dict(mask_window=3, team_warps=4)):
            assert (run(rps_mod, w, b, x0, w.steps, kernel=3, store_mode=store_mode, **opts) == ref).all(), opts
        pieces = [(0, 64_000), (64_000, 100_032), (164_032, w.d - 164_032)]
        parts = [run(rps_mod, w, b, x0, w.steps, shard=piece, kernel=3, store_mode=store_mode) for piece in pieces]
        assert (np.concatenate(parts, axis=1) == ref).all()


@pytest.mark.parametrize("n,d", [(5, 70_003), (8, 262_144), (17, 4097), (33, 20_011), (48, 50_001), (64, 300_007)])
def test_ring_gradient_averaging_matches_the_oracle(rps_mod, oracle, n, d):
    """Section 5's comparison method in the ring form (x is read a second time from the tile after the average,
    and the tile is handed back only then): against the oracle, and bit for bit across teams and ring depths."""
    w = wl.Workload("ring", n=n, d=d, dtype="bf16", p=0.2, gamma=0.05, sigma=0.1, seed=900 + n, steps=5, hetero=True)
    b = wl.make_targets(w)
    x0 = wl.f32_to_bf16_bits(np.random.default_rng(n * 7 + 1).standard_normal((n, d)).astype(np.float32))
    want = x0.copy()
    oracle.run(want, b, dtype="bf16", gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=3, steps=w.steps,
               average_gradients=True)
    ref = run(rps_mod, w, b, x0, w.steps, t0=3, kernel=3, average_gradients=True)
    g, o = wl.as_float64(w, ref), wl.as_float64(w, want)
    assert (np.abs(g - o) / (1 + np.abs(o))).max() <= BF16_TOL
    for team_warps, stages, traversal in ((1, 2, 0), (4, 3, 1), (8, 2, 0), (16, 0, 1), (3, 5, 0)):
        got = run(rps_mod, w, b, x0, w.steps, t0=3, kernel=3, average_gradients=True, team_warps=team_warps,
                  stages=stages, traversal=traversal)
        assert (got == ref).all(), (team_warps, stages, traversal)
    # the library's own choice for this step: the same kernel, except the streamed one where this kernel's lane
    # groups of 8, 16, 32 or 64 workers would be at most four fifths full (from 9 workers on)
    padded = 8
    while padded < n:
        padded *= 2
    if n >= 9 and 5 * n <= 4 * padded:
        ref = run(rps_mod, w, b, x0, w.steps, t0=3, kernel=4, average_gradients=True)
    assert (run(rps_mod, w, b, x0, w.steps, t0=3, average_gradients=True) == ref).all()


def test_steps_the_ring_is_not_built_for_run_as_the_staged_kernel(rps_mod, oracle):
    """fp32 replicas, few workers and tracked steps are not built in the ring form: asking for kernel 3 must still
    give the right step (gradient averaging is built: it runs as the ring kernel)."""
    for n, dtype, extra in ((8, "f32", {}), (3, "bf16", {}), (16, "bf16", dict(average_gradients=True))):
        w = wl.Workload("ring", n=n, d=30_011, dtype=dtype, p=0.2, gamma=0.1, sigma=0.1, seed=5, steps=3)
        b = wl.make_targets(w)
        x0 = wl.make_initial(w)
        want = x0.copy()
        oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps,
                   average_gradients=bool(extra))
        got = run(rps_mod, w, b, x0, w.steps, kernel=3, **extra)
        g, o = wl.as_float64(w, got), wl.as_float64(w, want)
        assert (np.abs(g - o) / (1 + np.abs(o))).max() <= (BF16_TOL if dtype == "bf16" else 1e-5)
    w = wl.Workload("ring", n=16, d=30_011, dtype="bf16", p=0.2, gamma=0.1, sigma=0.1, seed=5, steps=3)
    b = wl.make_targets(w)
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype="bf16", sigma=w.sigma, kernel=3)
    r.set_targets(b)
    r.track(3)
    r.step_n(3)
    tracked, trace = r.read(), r.read_trace()
    r.close()
    # tracked steps run in another lane shape (another summation order): equal within the tolerance, not bitwise
    g, o = wl.as_float64(w, tracked), wl.as_float64(w, run(rps_mod, w, b, wl.make_initial(w), 3, kernel=3))
    assert (np.abs(g - o) / (1 + np.abs(o))).max() <= BF16_TOL and np.isfinite(trace).all()


@pytest.mark.parametrize("store_mode", [1, 2, 3])
def test_a_ring_wait_that_runs_out_is_reported_and_harmless(rps_mod, store_mode):
    """Nothing is copied, so every warp's wait for its first tile runs out after the shortened limit: the kernel
    ends by itself, x is untouched, the next read reports it, and the device is as usable as before."""
    w = wl.Workload("ring", n=64, d=40_002, dtype="bf16", p=0.1, gamma=0.1, sigma=0.1, seed=9, steps=1)
    b = wl.make_targets(w)
    x0 = wl.f32_to_bf16_bits(np.random.default_rng(1).standard_normal((w.n, w.d)).astype(np.float32))
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype="bf16", sigma=w.sigma, kernel=3, wait_limit_ms=20,
                    store_mode=store_mode, withhold_copies=True)
    r.set_targets(b)
    r.write(x0)
    r.step()
    with pytest.raises(rps_mod.RPSError) as err:
        r.read()
    assert err.value.code == rps_mod.RPS_ECUDA and "gave up" in str(err.value)
    torch.cuda.synchronize()
    assert (r.x_dev[:, :w.d].view(torch.int16).cpu().numpy().view(np.uint16) == x0.view(np.uint16)).all()
    r.close()
    got = run(rps_mod, w, b, x0, 1, kernel=3, wait_limit_ms=20, store_mode=store_mode)
    assert (got == run(rps_mod, w, b, x0, 1, kernel=2, workers_per_lane=8, store_mode=1)).all()
