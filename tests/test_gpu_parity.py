"""Parity of the CUDA path (through the C ABI) with the CPU oracle.

Bars: drop masks, receive counts and servers bit-exact; fp32 replicas within
|delta| <= 1e-6 * (1 + |x|) after one step and 1e-5 (element-wise against
1 + |x|, and relative in the 2-norm) after T steps; bf16 replicas within 1e-2.
Every expected value comes from the oracle, which is given the same seeded
inputs and never sees a value computed on the GPU.
"""
import itertools

import numpy as np
import pytest
import torch

from paper_1810_07766_b200 import workloads as wl

pytestmark = pytest.mark.gpu

STEP_TOL = 1e-6
RUN_TOL = 1e-5
BF16_TOL = 1e-2


@pytest.fixture(scope="module")
def rps_mod():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_1810_07766_b200 import binding, build

    build.build()
    binding.load_library()
    return binding


def make(rps_mod, w, **kw):
    args = dict(dtype=w.dtype, sigma=w.sigma)
    args.update(kw)
    p = args.pop("p", w.p)
    return rps_mod.RPS(w.n, w.d, p, w.gamma, w.seed, **args)


def assert_close(w, got, want, tol):
    g, o = wl.as_float64(w, got), wl.as_float64(w, want)
    err = np.abs(g - o) / (1.0 + np.abs(o))
    assert err.max() <= tol, f"max |delta|/(1+|x|) = {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"
    rel = np.linalg.norm(g - o) / max(np.linalg.norm(o), 1e-30)
    assert rel <= tol, f"relative 2-norm error {rel:.3e}"
    return err.max()


# reduced-d twins of the five workloads: same n, p, gamma, sigma, seed; d ~ 1e5 with the
# same residues d % 4 and ceil(d/n) % 4 as the full size, so the same code paths run
TWINS = {
    "cfg1": wl.WORKLOADS["cfg1"],
    "cfg2": wl.WORKLOADS["cfg2"].scaled(d=100_010, steps=50),
    "cfg3": wl.WORKLOADS["cfg3"].scaled(d=100_008, steps=40),
    "cfg4": wl.WORKLOADS["cfg4"].scaled(d=100_005, steps=25),
    "cfg5": wl.WORKLOADS["cfg5"].scaled(d=65_536, steps=20),
}


def test_twins_keep_the_residues():
    for name, twin in TWINS.items():
        full = wl.WORKLOADS[name]
        assert twin.d % 4 == full.d % 4
        assert (-(-twin.d // twin.n)) % 4 == (-(-full.d // full.n)) % 4


# ------------------------------------------------------------------ masks: bit-exact

@pytest.mark.parametrize("n", [1, 2, 3, 4, 8, 16, 31, 32, 33, 64])
def test_masks_bit_exact(rps_mod, oracle, n):
    for p, sd, assign in itertools.product((0.0, 0.01, 0.05, 0.1, 0.2, 0.3, 0.999, 1.0), (True, False), (0, 1)):
        r = rps_mod.RPS(n, 1000, p, 0.1, 0xDEADBEEF12345678 ^ n, self_delivery=sd, assign=assign)
        for t in (0, 1, 2, 49, 199, (1 << 32) - 1, 1 << 32, (1 << 63) + 5):
            got = r.read_masks(t)
            want = oracle.masks(n, p, 0xDEADBEEF12345678 ^ n, t, self_delivery=sd, assign=assign)
            for a, b_ in zip(got, want):
                assert (a == b_).all(), (n, p, sd, assign, t)
        r.close()


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_masks_of_every_step_of_every_workload(rps_mod, oracle, name):
    w = wl.WORKLOADS[name]
    for p in (w.p_sweep or (w.p,)):
        r = rps_mod.RPS(w.n, 4096, p, w.gamma, w.seed, dtype=w.dtype)
        for t in range(w.steps):
            got = r.read_masks(t)
            want = oracle.masks(w.n, p, w.seed, t)
            assert all((a == b_).all() for a, b_ in zip(got, want))
        r.close()


# ------------------------------------------------------------------ noise

def test_gradient_noise_matches_the_oracle(rps_mod, oracle):
    """x = b = 0, gamma = sigma = 1, p = 1 gives x_1 = -xi: the raw noise field."""
    n, d = 8, 200_003
    w = wl.Workload("noise", n=n, d=d, dtype="f32", p=1.0, gamma=1.0, sigma=1.0, seed=12345, steps=1)
    for t in (0, 7, 1 << 33):
        r = make(rps_mod, w)
        r.set_step(t)
        r.step()
        got = r.read()
        want = np.zeros((n, d), dtype=np.float32)
        oracle.step(want, np.zeros((n, d), dtype=np.float32), dtype="f32", gamma=1.0, sigma=1.0, p=1.0, seed=w.seed, t=t)
        err = np.abs(got.astype(np.float64) - want)
        # approximate log2 / sqrt / sin / cos: absolute error of xi stays below 1e-4 even at the
        # smallest radii (where the log loses relative accuracy), and is ~1e-6 typically
        assert err.max() < 1e-4, err.max()
        assert np.median(err) < 2e-6
        assert abs(got.std() - 1.0) < 5e-3 and abs(got.mean()) < 5e-3
        r.close()


# ------------------------------------------------------------------ one step from a common state

@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_single_step_parity(rps_mod, oracle, name):
    w = TWINS[name]
    b = wl.make_targets(w)
    # a state in the middle of a run, produced by the oracle alone
    x0 = wl.make_initial(w)
    oracle.run(x0, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=3)
    for p in (w.p_sweep or (w.p,)):
        r = make(rps_mod, w, p=p)
        r.set_targets(b)
        for t in (3, 4):
            r.write(x0)
            r.set_step(t)
            r.step()
            got = r.read()
            want = x0.copy()
            oracle.step(want, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=p, seed=w.seed, t=t)
            assert_close(w, got, want, BF16_TOL if w.dtype == "bf16" else STEP_TOL)
            if w.dtype == "bf16":
                # rounding to bf16 may differ by one ulp where fp32 and fp64 sums straddle a tie
                assert (got != want).mean() < 0.02
        assert r.launch_count() >= 2
        r.close()


# ------------------------------------------------------------------ T free-running steps

@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_free_running_parity(rps_mod, oracle, name):
    w = TWINS[name]
    b = wl.make_targets(w)
    want = wl.make_initial(w)
    oracle.run(want, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
    r = make(rps_mod, w)
    r.set_targets(b)
    r.write(wl.make_initial(w))
    r.step_n(w.steps)
    assert r.get_step() == w.steps
    got = r.read()
    assert_close(w, got, want, BF16_TOL if w.dtype == "bf16" else RUN_TOL)
    # diagnostics against the oracle's, on the oracle's state
    r.write(want)
    dist2, cons = r.diag()
    o_dist2, o_cons = oracle.diag(want, b, dtype=w.dtype)
    assert dist2 == pytest.approx(o_dist2, rel=1e-9) and cons == pytest.approx(o_cons, rel=1e-9)
    r.close()


def test_mask_window_does_not_change_results(rps_mod):
    w = TWINS["cfg2"].scaled(d=10_010, steps=12)
    b = wl.make_targets(w)
    outs = []
    for window in (1, 5, 32):
        r = make(rps_mod, w, mask_window=window)
        r.set_targets(b)
        r.step_n(w.steps)
        outs.append(r.read())
        r.close()
    assert (outs[0] == outs[1]).all() and (outs[0] == outs[2]).all()


def test_resume_from_read_write_set_step(rps_mod):
    w = TWINS["cfg4"].scaled(d=20_005, steps=10)
    b = wl.make_targets(w)
    r = make(rps_mod, w)
    r.set_targets(b)
    r.step_n(10)
    straight = r.read()
    r.close()
    r = make(rps_mod, w)
    r.set_targets(b)
    r.step_n(4)
    mid = r.read()
    r.close()
    r = make(rps_mod, w)
    r.set_targets(b)
    r.write(mid)
    r.set_step(4)
    r.step_n(6)
    assert (r.read() == straight).all()
    r.close()


# ------------------------------------------------------------------ closed forms and invariants on the GPU output

def test_p0_and_p1_closed_forms(rps_mod):
    w = wl.WORKLOADS["cfg1"].scaled(d=4099)
    b = wl.make_targets(w)
    g = float(np.float32(w.gamma))
    r = make(rps_mod, w, p=0.0, sigma=0.0)
    r.set_targets(b)
    r.step_n(30)
    x = r.read()
    assert (x == x[0]).all()
    assert np.abs(x[0] - (1 - (1 - g) ** 30) * b.astype(np.float64).mean(axis=0)).max() <= 2e-6
    r.close()
    r = make(rps_mod, w, p=1.0, sigma=0.0)
    r.set_targets(b)
    r.step_n(30)
    assert np.abs(r.read() - (1 - (1 - g) ** 30) * b.astype(np.float64)).max() <= 2e-6
    r.close()


def test_receivers_hold_identical_values_and_outputs_are_convex(rps_mod, oracle):
    w = TWINS["cfg4"].scaled(d=9_001)
    b = wl.make_targets(w)
    x0 = np.random.default_rng(0).standard_normal(b.shape).astype(np.float32)
    r = make(rps_mod, w, sigma=0.0)
    r.set_targets(b)
    r.write(x0)
    r.step()
    x = r.read()
    _, down, _, _ = oracle.masks(w.n, w.p, w.seed, 0)
    block = -(-w.d // w.n)
    v = x0.astype(np.float64) - float(np.float32(w.gamma)) * (x0.astype(np.float64) - b)
    assert (x <= v.max(axis=0) + 1e-6).all() and (x >= v.min(axis=0) - 1e-6).all()
    for j in range(w.n):
        rows = [i for i in range(w.n) if (int(down[j]) >> i) & 1]
        cols = slice(j * block, min((j + 1) * block, w.d))
        assert (x[rows, cols] == x[rows[0], cols]).all()
    r.close()


# ------------------------------------------------------------------ forced masks: every drop pattern on tiny n

@pytest.mark.parametrize("n", [2, 3])
def test_forced_masks_every_pattern(rps_mod, oracle, n):
    d = 2 * n + 1
    rng = np.random.default_rng(n)
    b = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    r = rps_mod.RPS(n, d, 0.5, 0.25, 1)
    r.set_targets(b)
    words = range(1 << n)
    for up0, down0, up1 in itertools.product(words, words, words):
        up = np.array([up0, up1] + [up0] * (n - 2), dtype=np.uint64)
        down = np.array([down0, down0 ^ 1] + [down0] * (n - 2), dtype=np.uint64)
        r.write(x0)
        r.step_forced(up, down)
        got = r.read()
        want = x0.copy()
        oracle.step(want, b, dtype="f32", gamma=0.25, sigma=0.0, p=0.5, seed=1, t=0, forced_up=up, forced_down=down)
        assert np.abs(got.astype(np.float64) - want).max() <= STEP_TOL * (1 + np.abs(want).max())
    with pytest.raises(rps_mod.RPSError):
        r.step_forced(np.array([1 << n] * n, dtype=np.uint64), np.zeros(n, dtype=np.uint64))
    r.close()


# ------------------------------------------------------------------ edge shapes

EDGES = [
    # n, d, dtype
    (1, 1, "f32"), (1, 1000, "f32"), (2, 1, "f32"), (7, 3, "f32"), (5, 5, "f32"), (3, 2, "f32"),
    (64, 7, "f32"), (64, 64, "f32"), (64, 4099, "f32"), (33, 1025, "f32"), (17, 4097, "f32"),
    (9, 130, "f32"), (4, 31, "f32"), (4, 33, "f32"), (12, 127, "f32"), (3, 100_001, "f32"),
    (1, 9, "bf16"), (6, 3, "bf16"), (8, 1031, "bf16"), (16, 4097, "bf16"), (33, 2050, "bf16"), (64, 8191, "bf16"),
]


@pytest.mark.parametrize("n,d,dtype", EDGES)
def test_edge_shapes(rps_mod, oracle, n, d, dtype):
    w = wl.Workload("edge", n=n, d=d, dtype=dtype, p=0.3, gamma=0.1, sigma=0.1, seed=100 + n, steps=3)
    b = wl.make_targets(w)
    for sd, assign in ((True, 0), (False, 0), (True, 1)):
        want = wl.make_initial(w)
        oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps,
                   self_delivery=sd, assign=assign)
        for kernel, copy_mode, slice_bytes, store_mode in ((1, 0, 0, 0), (2, 1, 0, 1), (2, 2, 0, 2), (2, 0, 8, 2),
                                                            (2, 1, 0, 2), (2, 0, 0, 3), (2, 0, 8, 3)):
            if slice_bytes == 8 and dtype != "bf16":
                continue
            r = make(rps_mod, w, self_delivery=sd, assign=assign, kernel=kernel, copy_mode=copy_mode,
                     slice_bytes=slice_bytes, store_mode=store_mode)
            r.set_targets(b)
            r.x_dev[:, d:] = 3.0         # sentinel in the padding between d and the row pitch
            r.step_n(w.steps)
            got = r.read()
            assert_close(w, got, want, BF16_TOL if dtype == "bf16" else 3 * STEP_TOL)
            # padding is left alone, except that the columns sharing a 16-byte unit with the last
            # real column may be zeroed
            unit = 4 if dtype == "f32" else 8
            edge = -(-d // unit) * unit
            assert (r.x_dev[:, edge:].float() == 3.0).all()
            shared_unit = r.x_dev[:, d:edge].float()
            assert ((shared_unit == 3.0) | (shared_unit == 0.0)).all()
            r.close()


# every shape of the fused kernel computes the same step:
# (kernel, workers_per_lane, stages, consumer_warps, copy_mode, slice_bytes, store_mode)
VARIANTS = [(1, 0, 0, 0, 0, 0, 0), (1, 4, 0, 0, 0, 0, 0), (2, 0, 0, 0, 0, 0, 0), (2, 2, 0, 0, 1, 0, 1),
            (2, 4, 2, 4, 2, 0, 2), (2, 8, 4, 3, 1, 0, 2), (2, 4, 5, 16, 2, 0, 1), (2, 2, 8, 1, 2, 0, 2),
            (2, 8, 2, 8, 2, 0, 1), (2, 4, 3, 5, 1, 0, 2), (2, 8, 2, 12, 1, 0, 1), (2, 8, 2, 20, 2, 8, 2),
            (2, 8, 3, 7, 1, 8, 1), (2, 4, 2, 16, 0, 0, 2), (2, 8, 2, 8, 0, 0, 2), (2, 8, 2, 12, 0, 0, 3),
            (2, 4, 2, 16, 0, 0, 3), (2, 8, 3, 5, 0, 8, 3), (2, 2, 2, 3, 1, 0, 3)]


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_kernel_variants(rps_mod, oracle, name):
    w = TWINS[name].scaled(d=TWINS[name].d // 2 + (3 if name != "cfg5" else 0), steps=3)
    b = wl.make_targets(w)
    want = wl.make_initial(w)
    oracle.run(want, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
    for kernel, wpt, stages, warps, copy_mode, slice_bytes, store_mode in VARIANTS:
        r = make(rps_mod, w, kernel=kernel, workers_per_lane=wpt, stages=stages, consumer_warps=warps,
                 copy_mode=copy_mode, slice_bytes=slice_bytes, store_mode=store_mode)
        r.set_targets(b)
        r.step_n(w.steps)
        got = r.read()
        assert_close(w, got, want, BF16_TOL if w.dtype == "bf16" else 3 * STEP_TOL)
        r.close()


def test_guard_bands_around_device_buffers(rps_mod):
    """The kernels stay inside [n][pitch]: a sentinel pattern placed in the scratch tail and in
    the targets' padding is intact after stepping."""
    w = TWINS["cfg4"].scaled(d=50_001, steps=5)
    r = make(rps_mod, w)
    r.set_targets(wl.make_targets(w))
    r.b_dev[:, w.d:] = 7.0
    tail = r.scratch[-128:].clone()
    r.step_n(w.steps)
    torch.cuda.synchronize()
    assert (r.b_dev[:, w.d:] == 7.0).all()
    assert (r.scratch[-128:] == tail).all()
    assert not r.x_dev[:, w.d:].any()
    r.read()                              # also checks the kernels' error word
    r.close()


# ------------------------------------------------------------------ host-buffer step

def test_step_host_equals_resident_step(rps_mod):
    w = TWINS["cfg2"].scaled(d=30_002, steps=4)
    b = wl.make_targets(w)
    r = make(rps_mod, w)
    r.set_targets(b)
    r.step_n(w.steps)
    want = r.read()
    r.close()
    r = make(rps_mod, w)
    x_host = torch.zeros((w.n, w.d), dtype=torch.float32).pin_memory()
    b_host = torch.from_numpy(b).pin_memory()
    for _ in range(w.steps):
        r.step_host(x_host, b_host)
    assert (x_host.numpy() == want).all()
    r.close()


@pytest.mark.parametrize("n,d,dtype", [(8, 600_011, "f32"), (64, 200_000, "bf16"), (16, 2_000_003, "f32")])
def test_step_host_in_pieces_equals_resident_step(rps_mod, oracle, n, d, dtype):
    """Large enough for the host-buffer step to go through in several pieces of columns (upload, step and
    download overlapped): bit for bit the resident step, with and without uploading the targets every step,
    tracked steps included; and within the step's tolerance of the oracle."""
    w = wl.Workload("pieces", n=n, d=d, dtype=dtype, p=0.1, gamma=0.05, sigma=0.1, seed=40 + n, steps=3)
    b = wl.make_targets(w)
    bits = np.uint16 if dtype == "bf16" else np.uint32
    r = make(rps_mod, w, kernel=2)
    r.set_targets(b)
    r.track(w.steps)
    r.step_n(w.steps)
    want = r.read()
    want_trace = r.read_trace()
    r.close()
    tdtype = torch.float32 if dtype == "f32" else torch.int16
    for resident_targets in (False, True):
        r = make(rps_mod, w, kernel=2)
        r.track(w.steps)
        x_host = torch.zeros((n, d), dtype=tdtype).pin_memory()
        b_host = torch.from_numpy(b if dtype == "f32" else b.view(np.int16)).pin_memory()
        if resident_targets:
            r.set_targets(b)
        for _ in range(w.steps):
            r.step_host(x_host, None if resident_targets else b_host)
        assert r.get_step() == w.steps
        got = x_host.numpy().view(bits)
        assert (got == want.view(bits)).all()
        assert (r.read().view(bits) == want.view(bits)).all()
        assert np.allclose(r.read_trace(), want_trace, rtol=1e-9)
        r.close()
    ref = wl.make_initial(w)
    oracle.run(ref, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
    assert_close(w, want, ref, BF16_TOL if dtype == "bf16" else 3 * STEP_TOL)


def test_profile_counts_launches(rps_mod):
    w = TWINS["cfg1"]
    r = make(rps_mod, w, mask_window=4)
    r.profile(True)
    r.step_n(8)
    fused_ms, fused_n, mask_ms, mask_n = r.profile_read()
    assert (fused_n, mask_n) == (8, 2) and fused_ms > 0 and mask_ms > 0
    r.profile(False)
    assert r.launch_count() == 10
    r.close()


# ------------------------------------------------------------------ full sizes, sampled columns

def sampled_columns(w, rng, count=4096):
    """Random columns plus the first and last few columns of every block and of the row."""
    block = -(-w.d // w.n)
    edges = [0, 1, 2, 3, w.d - 4, w.d - 3, w.d - 2, w.d - 1]
    for j in range(1, w.n):
        for off in (-5, -4, -3, -2, -1, 0, 1, 2, 3, 4):
            edges.append(j * block + off)
    cols = np.concatenate([rng.integers(0, w.d, size=count), np.array(edges)])
    return np.unique(cols[(cols >= 0) & (cols < w.d)]).astype(np.int64)


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_size_sampled_columns(rps_mod, oracle, name):
    """The workload at its full size, in the launch configuration the benchmark times (library
    defaults): T = 3 free-running steps, checked on sampled columns that the oracle recomputes
    from the same inputs (columns evolve independently of one another)."""
    w = wl.WORKLOADS[name]
    steps = 3
    b = wl.make_targets(w)
    cols = sampled_columns(w, np.random.default_rng(w.seed))
    want = np.ascontiguousarray(wl.make_initial(w)[:, cols])
    b_cols = np.ascontiguousarray(b[:, cols])
    for t in range(steps):
        oracle.step_columns(w.d, cols, want, b_cols, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=t)
    r = make(rps_mod, w)
    r.set_targets(b)
    del b
    r.step_n(steps)
    got = r.read()[:, cols]
    assert_close(w, got, want, BF16_TOL if w.dtype == "bf16" else 3 * STEP_TOL)
    for t in range(steps):
        assert all((a == o).all() for a, o in zip(r.read_masks(t), oracle.masks(w.n, w.p, w.seed, t)))
    r.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_size_whole_run_sampled_columns(rps_mod, oracle, name):
    """The workload at its full size for its whole run (50, 200, 50 and 100 steps), every drop probability of
    its sweep, library defaults, free-running from x = 0: the sampled columns against the oracle's own run of
    those columns, within the T-step bar.  cfg3 runs tracked, as its description asks (distance to the optimum
    at every step): the trace must be what rps_diag measures on the final state, and must have come down."""
    w0 = wl.WORKLOADS[name]
    b = wl.make_targets(w0)
    cols = sampled_columns(w0, np.random.default_rng(w0.seed + 1000), count=2048)
    b_cols = np.ascontiguousarray(b[:, cols])
    tracked = name == "cfg3"
    for p in (w0.p_sweep or (w0.p,)):
        want = np.ascontiguousarray(wl.make_initial(w0)[:, cols])
        for t in range(w0.steps):
            oracle.step_columns(w0.d, cols, want, b_cols, dtype=w0.dtype, gamma=w0.gamma, sigma=w0.sigma, p=p,
                                seed=w0.seed, t=t)
        r = make(rps_mod, w0, p=p)
        r.set_targets(b)
        if tracked:
            r.track(w0.steps)
        r.step_n(w0.steps)
        got = r.read()[:, cols]
        assert r.get_step() == w0.steps
        assert_close(w0, got, want, BF16_TOL if w0.dtype == "bf16" else RUN_TOL)
        if tracked:
            trace = r.read_trace()
            dist2, cons = r.diag()
            assert np.allclose(trace[-1], (dist2, cons), rtol=1e-4)
            assert trace[-1][0] < 0.01 * trace[0][0] and np.isfinite(trace).all()
        r.close()
    del b
    torch.cuda.empty_cache()


# ------------------------------------------------------------------ every element: laps of the rings, full sizes

@pytest.mark.parametrize("n,d,dtype", [(8, 3_000_011, "f32"), (16, 2_400_003, "f32"), (32, 2_000_037, "f32"),
                                       (32, 1_500_007, "bf16"), (64, 1_048_584, "bf16")])
def test_default_shapes_lap_their_rings_every_element(rps_mod, oracle, n, d, dtype):
    """The library's own choice of kernel for each kind of workload (staged with 4 and with 8 workers per lane,
    the ring kernel, the streamed kernel) on a model long enough that every CTA takes a dozen or more tiles, so
    that every stage of its ring is reused many times: three free-running steps, which walk the columns up, down
    and up again, compared with the oracle's run in EVERY element."""
    w = wl.Workload("laps", n=n, d=d, dtype=dtype, p=0.1, gamma=0.05, sigma=0.1, seed=4321 + n, steps=3)
    b = wl.make_targets(w)
    want = wl.make_initial(w)
    oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
    r = make(rps_mod, w)
    r.set_targets(b)
    r.step_n(w.steps)
    got = r.read()
    r.close()
    assert_close(w, got, want, BF16_TOL if dtype == "bf16" else 3 * STEP_TOL)


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_size_one_step_every_element(rps_mod, oracle, name):
    """One step of the workload at its full size from a state in which every replica differs (worker i starts
    from the targets of worker n-1-i), library defaults: the WHOLE state against the oracle's step, row by row."""
    w = wl.WORKLOADS[name]
    b = wl.make_targets(w)
    x0 = np.ascontiguousarray(b[::-1])
    want = x0.copy()
    oracle.step(want, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=7)
    r = make(rps_mod, w)
    r.set_targets(b)
    r.write(x0)
    del x0, b
    r.set_step(7)
    r.step()
    got = r.read()
    r.close()
    tol = BF16_TOL if w.dtype == "bf16" else STEP_TOL
    worst = 0.0
    for i in range(w.n):  # a row at a time keeps the fp64 copies small
        g, o = wl.as_float64(w, got[i:i + 1]), wl.as_float64(w, want[i:i + 1])
        worst = max(worst, float((np.abs(g - o) / (1.0 + np.abs(o))).max()))
    assert worst <= tol, worst
    torch.cuda.empty_cache()


# ------------------------------------------------------------------ bounded waits

@pytest.mark.parametrize("store_mode", [1, 2, 3])
def test_a_wait_that_runs_out_is_reported_and_harmless(rps_mod, store_mode):
    """The staged kernel's waits are bounded.  With the copies withheld nothing ever lands, every compute
    warp gives up after the (shortened) limit, the kernel ends by itself, the replicas are untouched, the
    next read reports the error, and the device is as usable as before."""
    w = TWINS["cfg2"].scaled(d=40_002, steps=1)
    b = wl.make_targets(w)
    x0 = np.random.default_rng(1).standard_normal(b.shape).astype(np.float32)
    r = make(rps_mod, w, kernel=2, store_mode=store_mode, wait_limit_ms=20, withhold_copies=True)
    r.set_targets(b)
    r.write(x0)
    r.step()
    with pytest.raises(rps_mod.RPSError) as err:
        r.read()
    assert err.value.code == rps_mod.RPS_ECUDA and "gave up" in str(err.value)
    torch.cuda.synchronize()
    assert (r.x_dev[:, :w.d].cpu().numpy() == x0).all()
    r.close()
    # the same handle settings without the test aid work, on the same device, right after
    r = make(rps_mod, w, kernel=2, store_mode=store_mode, wait_limit_ms=20)
    r.set_targets(b)
    r.write(x0)
    r.step()
    assert np.isfinite(r.read()).all()
    r.close()


# ------------------------------------------------------------------ gradient averaging (Section 5's comparison)

@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg4", "cfg5"])
def test_gradient_averaging_parity(rps_mod, oracle, name):
    w = TWINS[name].scaled(d=TWINS[name].d // 2 + (1 if name != "cfg5" else 0), steps=6)
    b = wl.make_targets(w)
    want = wl.make_initial(w)
    oracle.run(want, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps,
               average_gradients=True)
    tol = BF16_TOL if w.dtype == "bf16" else 6 * STEP_TOL
    for kernel, store_mode, copy_mode in ((0, 0, 0), (1, 0, 0), (2, 1, 1), (2, 2, 2), (2, 3, 0)):
        r = make(rps_mod, w, average_gradients=True, kernel=kernel, store_mode=store_mode, copy_mode=copy_mode)
        r.set_targets(b)
        r.step_n(w.steps)
        assert_close(w, r.read(), want, tol)
        r.close()
    # and it is a different method: model averaging from the same inputs ends elsewhere
    r = make(rps_mod, w)
    r.set_targets(b)
    r.step_n(w.steps)
    other = r.read()
    r.close()
    assert np.abs(wl.as_float64(w, other) - wl.as_float64(w, want)).max() > 1e-3


# ------------------------------------------------------------------ cache-related options change no bit

def test_traversal_and_l2_policy_do_not_change_results(rps_mod):
    """Walking the columns downwards on odd steps, hinting the L2 cache, or letting a launch be set up while the
    one before it drains, only moves work in time."""
    for dtype, n, d in (("f32", 8, 300_010), ("f32", 32, 100_005), ("bf16", 64, 65_536)):
        w = wl.Workload("cache", n=n, d=d, dtype=dtype, p=0.1, gamma=0.05, sigma=0.1, seed=11, steps=5)
        b = wl.make_targets(w)
        out = []
        for kernel, traversal, l2_policy, overlap in ((2, 0, 0, 0), (2, 1, 1, 1), (2, 0, 2, 2), (2, 1, 2, 2),
                                                       (2, 0, 0, 2), (1, 0, 0, 0), (1, 1, 0, 2)):
            r = make(rps_mod, w, kernel=kernel, workers_per_lane=4, traversal=traversal, l2_policy=l2_policy,
                     launch_overlap=overlap)
            r.set_targets(b)
            r.step_n(w.steps)
            out.append(r.read().view(np.uint16 if dtype == "bf16" else np.uint32))
            r.close()
        for other in out[1:]:
            assert (other == out[0]).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("workers_per_lane,n,warps", [(2, 24, 4), (2, 31, 16), (2, 32, 8), (4, 33, 16), (4, 64, 4),
                                                      (4, 64, 16)])
def test_staged_lane_groups_of_sixteen_lanes(rps_mod, oracle, dtype, workers_per_lane, n, warps):
    """The widest lane groups of the staged kernel (16 lanes: 2 workers per lane with more than 16 workers, 4 with
    more than 32; a warp is then only 8 fp32 columns wide) in every way of filling and emptying a stage, whole and
    as a shard, against the oracle: every element, and twice (a stage read before it had landed shows only in the
    first tiles of a CTA and not in every run)."""
    d = 70_003
    w = wl.Workload("wide", n=n, d=d, dtype=dtype, p=0.2, gamma=0.05, sigma=0.1, seed=60 + n, steps=2, hetero=True)
    b = wl.make_targets(w)
    x0 = np.random.default_rng(n).standard_normal((n, d)).astype(np.float32)
    if dtype == "bf16":
        x0 = wl.f32_to_bf16_bits(x0)
    want = x0.copy()
    oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=5, steps=w.steps)
    for store_mode, copy_mode, shard in ((0, 0, None), (1, 2, None), (2, 2, (11_072, 52_193)), (3, 0, None),
                                         (2, 1, (11_072, 52_193))):
        begin, cols = shard if shard else (0, d)
        for _ in range(2):
            r = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, kernel=2,
                            workers_per_lane=workers_per_lane, consumer_warps=warps, store_mode=store_mode,
                            copy_mode=copy_mode, shard_begin=begin if shard else 0, shard_cols=cols if shard else 0)
            r.set_targets(np.ascontiguousarray(b[:, begin:begin + cols]))
            r.write(np.ascontiguousarray(x0[:, begin:begin + cols]))
            r.set_step(5)
            r.step_n(w.steps)
            got = r.read()
            r.close()
            g = wl.as_float64(w, got)
            o = wl.as_float64(w, np.ascontiguousarray(want[:, begin:begin + cols]))
            err = (np.abs(g - o) / (1.0 + np.abs(o))).max()
            assert err <= (1e-2 if dtype == "bf16" else 1e-5), (store_mode, copy_mode, shard, float(err))
