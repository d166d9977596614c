"""The streamed-workers kernel (kernel 4: a lane walks all n workers of its 16-byte column slice in order, every
warp refills a ring of its own) against the oracle, element by element, on shapes that make every warp lap its
ring many times in both traversal directions, and against itself: warps, ring depth, traversal, launch mode,
mask window and column shards may not change one bit of x, and where the direct kernel sums in the same order
(all n workers in one lane: n <= 8) the two agree bit for bit."""
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


def run(rps_mod, w, b, x0, steps, t0=0, shard=None, strict_padding=True, **opts):
    begin, cols = shard if shard else (0, w.d)
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype=w.dtype, sigma=w.sigma,
                    shard_begin=begin if shard else 0, shard_cols=cols if shard else 0, **opts)
    r.set_targets(np.ascontiguousarray(b[:, begin:begin + cols]))
    r.write(np.ascontiguousarray(x0[:, begin:begin + cols]))
    r.x_dev[:, cols:] = 3.0  # sentinel in the padding between the last column and the row pitch
    r.set_step(t0)
    r.step_n(steps)
    got = r.read()
    # the streamed kernel writes no padding at all; the other kernels may zero what shares a 16-byte unit with the
    # last column
    edge = cols if strict_padding else -(-cols // 8) * 8
    assert (r.x_dev[:, edge:].float() == 3.0).all(), "padding was written"
    r.close()
    return got


def start(w, seed):
    x0 = np.random.default_rng(seed).standard_normal((w.n, w.d)).astype(np.float32)
    return wl.f32_to_bf16_bits(x0) if w.dtype == "bf16" else x0


def rel_err(w, got, want):
    g, o = wl.as_float64(w, got), wl.as_float64(w, want)
    return (np.abs(g - o) / (1 + np.abs(o))).max()


SHAPES = [
    # n, d: odd n (the last pair has one worker), n = 2, ragged d, d below one tile, blocks cut inside a slice
    (2, 50_001), (3, 4097), (5, 70_003), (8, 262_144), (9, 1031), (16, 131_075), (17, 40_970), (32, 65_536),
    (33, 20_011), (48, 50_001), (63, 8191), (64, 65_536), (64, 300_007), (64, 7), (6, 1), (7, 255), (4, 256),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,d", SHAPES)
def test_stream_matches_the_oracle_and_its_options_change_no_bit(rps_mod, oracle, dtype, n, d):
    w = wl.Workload("stream", n=n, d=d, dtype=dtype, p=0.2, gamma=0.05, sigma=0.1, seed=400 + n, steps=4, hetero=True)
    b = wl.make_targets(w)
    x0 = start(w, n * 7 + 1)
    want = x0.copy()
    oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=3, steps=w.steps)
    # blocks narrower than a lane's slice are not built in this form: such a step runs as the staged kernel
    covered = -(-d // n) >= (8 if dtype == "bf16" else 4)
    run_ = lambda *a, **k: run(*a, strict_padding=covered, **k)
    ref = run_(rps_mod, w, b, x0, w.steps, t0=3, kernel=4)
    assert rel_err(w, ref, want) <= (BF16_TOL if dtype == "bf16" else RUN_TOL)
    for warps, stages, team in ((1, 2, 1), (3, 5, 1), (8, 8, 2), (16, 0, 0), (24, 4, 8), (32, 3, 4), (32, 2, 16),
                                (12, 3, 4), (30, 2, 3)):
        got = run_(rps_mod, w, b, x0, w.steps, t0=3, kernel=4, consumer_warps=warps, stages=stages, team_warps=team)
        assert (got == ref).all(), (warps, stages, team, int((got != ref).sum()))
    for opts in (dict(traversal=1), dict(launch_overlap=1), dict(mask_window=1), dict(early_targets=1),
                 dict(early_targets=1, launch_overlap=1), dict(workers_per_lane=2),
                 dict(workers_per_lane=2, team_warps=4, consumer_warps=20, stages=6), dict(store_mode=2),
                 dict(store_mode=2, team_warps=4, consumer_warps=20, traversal=1)):
        if ("workers_per_lane" in opts or "store_mode" in opts) and not covered:
            continue  # (the staged kernel takes these options as its lane shape and tile, which set its summation order)
        assert (run_(rps_mod, w, b, x0, w.steps, t0=3, kernel=4, **opts) == ref).all(), opts
    if n <= 8 and covered:
        # the direct kernel with all workers in one lane adds them in the same order
        same_order = run(rps_mod, w, b, x0, w.steps, t0=3, kernel=1, workers_per_lane=8, strict_padding=False)
        assert (same_order == ref).all()


@pytest.mark.parametrize("self_delivery,assign,p", [(True, 1, 0.3), (False, 0, 0.6), (False, 1, 0.95), (True, 0, 0.0),
                                                    (True, 0, 1.0)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_stream_single_step_in_every_mask_mode(rps_mod, oracle, dtype, self_delivery, assign, p):
    """One step from a common state: random server assignment, every message droppable (blocks that nobody
    averages keep v everywhere), nothing dropped, everything dropped."""
    w = wl.Workload("stream", n=12, d=90_011, dtype=dtype, p=p, gamma=0.1, sigma=0.05, seed=31, steps=1)
    b = wl.make_targets(w)
    x0 = start(w, 3)
    for t in (0, 1, (1 << 32) - 1, 1 << 40):
        want = x0.copy()
        oracle.step(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=p, seed=w.seed, t=t,
                    self_delivery=self_delivery, assign=assign)
        got = run(rps_mod, w, b, x0, 1, t0=t, kernel=4, self_delivery=self_delivery, assign=assign)
        assert rel_err(w, got, want) <= (BF16_TOL if dtype == "bf16" else STEP_TOL), (t, rel_err(w, got, want))


@pytest.mark.parametrize("n", [2, 3])
def test_stream_forced_masks_every_pattern(rps_mod, oracle, n):
    """Every drop pattern of one block at n = 2, 3 (the other blocks fully delivered), against the oracle."""
    d = 3 * 128 * n + 5
    w = wl.Workload("stream", n=n, d=d, dtype="f32", p=0.5, gamma=0.1, sigma=0.1, seed=8, steps=1)
    b = wl.make_targets(w)
    x0 = start(w, 2)
    full = (1 << n) - 1
    r = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype="f32", sigma=w.sigma, kernel=4)
    r.set_targets(b)
    for j in range(n):
        for up_bits in range(1 << n):
            for down_bits in range(1 << n):
                up = np.full(n, full, dtype=np.uint64)
                down = np.full(n, full, dtype=np.uint64)
                up[j], down[j] = up_bits, down_bits
                want = x0.copy()
                oracle.step(want, b, dtype="f32", gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=5,
                            forced_up=up, forced_down=down)
                r.write(x0)
                r.set_step(5)
                r.step_forced(up, down)
                assert rel_err(w, r.read(), want) <= STEP_TOL, (j, up_bits, down_bits)
    r.close()


@pytest.mark.parametrize("average_gradients", [False, True])
def test_stream_shards_reproduce_the_whole_model(rps_mod, average_gradients):
    for dtype, n, d in (("bf16", 64, 200_017), ("f32", 10, 150_001)):
        w = wl.Workload("stream", n=n, d=d, dtype=dtype, p=0.1, gamma=0.02, sigma=0.1, seed=77, steps=5)
        b = wl.make_targets(w)
        x0 = start(w, 5)
        ref = run(rps_mod, w, b, x0, w.steps, kernel=4, average_gradients=average_gradients)
        pieces = [(0, 64_000), (64_000, 36_032), (100_032, d - 100_032)]
        parts = [run(rps_mod, w, b, x0, w.steps, shard=piece, kernel=4, average_gradients=average_gradients)
                 for piece in pieces]
        assert (np.concatenate(parts, axis=1) == ref).all()


@pytest.mark.parametrize("n,d,dtype,warps", [(8, 3_000_011, "f32", 0), (64, 1_048_584, "bf16", 6),
                                             (64, 600_007, "bf16", 0)])
def test_stream_laps_its_rings_many_times_every_element(rps_mod, oracle, n, d, dtype, warps):
    """Three free-running steps (up, down, up) on a model long enough that every warp takes several tiles, one
    after the other through its ring, and laps the ring dozens of times; every element against the oracle's run."""
    w = wl.Workload("stream", n=n, d=d, dtype=dtype, p=0.1, gamma=0.05, sigma=0.1, seed=1234 + n, steps=3)
    b = wl.make_targets(w)
    x0 = wl.make_initial(w)
    want = x0.copy()
    oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
    got = run(rps_mod, w, b, x0, w.steps, kernel=4, consumer_warps=warps, team_warps=2 if warps else 0)
    assert rel_err(w, got, want) <= (BF16_TOL if dtype == "bf16" else RUN_TOL)


def test_steps_the_stream_kernel_is_not_built_for_still_run(rps_mod, oracle):
    """One worker, blocks narrower than a lane's slice: asking for kernel 4 must still give the right step."""
    for n, d, dtype in ((1, 30_011, "f32"), (16, 100, "bf16")):
        w = wl.Workload("stream", n=n, d=d, dtype=dtype, p=0.2, gamma=0.1, sigma=0.1, seed=5, steps=3)
        b = wl.make_targets(w)
        x0 = wl.make_initial(w)
        want = x0.copy()
        oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
        got = run(rps_mod, w, b, x0, w.steps, kernel=4, strict_padding=False)
        assert rel_err(w, got, want) <= (BF16_TOL if dtype == "bf16" else RUN_TOL)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,d", [(2, 50_001), (3, 4097), (5, 70_003), (8, 262_144), (17, 40_970), (33, 20_011),
                                 (48, 50_001), (64, 300_007), (64, 7), (7, 255)])
def test_stream_gradient_averaging_matches_the_oracle(rps_mod, oracle, dtype, n, d):
    """Section 5's comparison method in the streamed form (the updates are summed, and a tile's rows of x go through
    the ring a second time for the receivers): against the oracle's run, and bit for bit across warps, teams, ring
    depths, traversal, launch mode and steps per launch; the padding stays untouched."""
    w = wl.Workload("stream", n=n, d=d, dtype=dtype, p=0.2, gamma=0.05, sigma=0.1, seed=700 + n, steps=7, hetero=True)
    b = wl.make_targets(w)
    x0 = start(w, n * 5 + 2)
    want = x0.copy()
    oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=3, steps=w.steps,
               average_gradients=True)
    covered = -(-d // n) >= (8 if dtype == "bf16" else 4)
    ref = run(rps_mod, w, b, x0, w.steps, t0=3, kernel=4, average_gradients=True, strict_padding=covered)
    assert rel_err(w, ref, want) <= (BF16_TOL if dtype == "bf16" else RUN_TOL)
    if not covered:
        return
    for opts in (dict(consumer_warps=1, team_warps=1, stages=2), dict(consumer_warps=16, stages=3, traversal=1),
                 dict(team_warps=2, consumer_warps=6, stages=5, launch_overlap=1), dict(fuse_steps=1),
                 dict(fuse_steps=2, mask_window=3), dict(early_targets=2, stages=8)):
        base = ref if "traversal" not in opts else run(rps_mod, w, b, x0, w.steps, t0=3, kernel=4,
                                                       average_gradients=True, traversal=1, fuse_steps=1)
        got = run(rps_mod, w, b, x0, w.steps, t0=3, kernel=4, average_gradients=True, **opts)
        assert (got == base).all(), (opts, int((got != base).sum()))
    # one step, forced to the other kernels' tolerance: the single-step bound
    one = x0.copy()
    oracle.run(one, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=3, steps=1,
               average_gradients=True)
    got = run(rps_mod, w, b, x0, 1, t0=3, kernel=4, average_gradients=True)
    assert rel_err(w, got, one) <= (BF16_TOL if dtype == "bf16" else STEP_TOL)


def test_a_stream_wait_that_runs_out_is_reported_and_harmless(rps_mod):
    """Nothing is copied, so every warp's wait for its first pair runs out after the shortened limit: the kernel
    ends by itself, x is untouched, the next read reports it, and the device is as usable as before."""
    w = wl.Workload("stream", n=64, d=40_960, dtype="bf16", p=0.1, gamma=0.1, sigma=0.1, seed=9, steps=1)
    b = wl.make_targets(w)
    x0 = start(w, 1)
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype="bf16", sigma=w.sigma, kernel=4, wait_limit_ms=20,
                    withhold_copies=True)
    r.set_targets(b)
    r.write(x0)
    r.step()
    with pytest.raises(rps_mod.RPSError) as err:
        r.read()
    assert err.value.code == rps_mod.RPS_ECUDA and "gave up" in str(err.value)
    torch.cuda.synchronize()
    assert (r.x_dev[:, :w.d].view(torch.int16).cpu().numpy().view(np.uint16) == x0.view(np.uint16)).all()
    r.close()
    assert (run(rps_mod, w, b, x0, 1, kernel=4, wait_limit_ms=20) == run(rps_mod, w, b, x0, 1, kernel=4)).all()


TRACE_RTOL = 1e-4


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,d,self_delivery,p", [(2, 50_001, True, 0.3), (5, 70_003, True, 0.2), (17, 40_970, False, 0.7),
                                                 (48, 50_001, True, 0.05), (64, 300_007, True, 0.1),
                                                 (64, 65_536, False, 0.95), (12, 90_011, True, 1.0), (9, 8_200, True, 0.0)])
def test_stream_tracked_steps_report_the_oracle_diagnostics(rps_mod, oracle, dtype, n, d, self_delivery, p):
    """Tracked steps in the streamed form: every entry of the trace against the oracle's diagnostics of the state
    that step left in memory (lanes on block boundaries and on the end of the row included, blocks that nobody
    averages, everything and nothing delivered), and tracking changes no bit of x."""
    w = wl.Workload("stream", n=n, d=d, dtype=dtype, p=p, gamma=0.1, sigma=0.1, seed=77 + n, steps=4, hetero=True)
    b = wl.make_targets(w)
    x0 = start(w, 9)
    untracked = run(rps_mod, w, b, x0, w.steps, kernel=4, self_delivery=self_delivery)
    for warps, team in ((0, 0), (16, 2), (5, 1)):
        r = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, kernel=4, self_delivery=self_delivery,
                        consumer_warps=warps, team_warps=team)
        r.set_targets(b)
        r.write(x0)
        r.track(w.steps)
        states = []
        for _ in range(w.steps):
            r.step()
            states.append(r.read())
        trace = r.read_trace()
        r.close()
        assert trace.shape == (w.steps, 2)
        for k, x in enumerate(states):
            dist2, cons = oracle.diag(x, b, dtype=dtype)
            assert abs(trace[k, 0] - dist2) <= TRACE_RTOL * dist2 + 1e-12 * n * d, (warps, k, trace[k, 0], dist2)
            assert abs(trace[k, 1] - cons) <= TRACE_RTOL * cons + 1e-12 * n * d, (warps, k, trace[k, 1], cons)
        assert (states[-1] == untracked).all()


@pytest.mark.parametrize("n,d,dtype", [(8, 300_010, "f32"), (16, 100_008, "f32"), (32, 100_005, "f32"), (64, 65_536, "bf16"),
                                       (3, 70_001, "bf16")])
def test_targets_copied_ahead_of_the_wait_change_no_bit(rps_mod, n, d, dtype):
    """The first stages' copies of b may be issued before a CTA waits for the step before it (early_targets):
    with them, without them, in a plain launch and with targets replaced between steps by the library's own
    upload, the staged and the streamed kernel give the same bits."""
    w = wl.Workload("early", n=n, d=d, dtype=dtype, p=0.1, gamma=0.05, sigma=0.1, seed=11, steps=6)
    b = wl.make_targets(w)
    b2 = wl.make_targets(wl.Workload("early", n=n, d=d, dtype=dtype, p=0.1, gamma=0.05, sigma=0.1, seed=12, steps=6))
    x0 = start(w, 4)
    for kernel in (2, 4):
        outs = []
        for opts in (dict(early_targets=1), dict(early_targets=2), dict(early_targets=2, launch_overlap=1), dict()):
            r = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, kernel=kernel, **opts)
            r.set_targets(b)
            r.write(x0)
            r.step_n(3)
            r.set_targets(b2)  # an upload between two steps: the next step's early copies must see it
            r.step_n(3)
            outs.append(r.read())
            r.close()
        for other in outs[1:]:
            assert (other == outs[0]).all(), kernel


@pytest.mark.parametrize("n,d,dtype", [(64, 300_007, "bf16"), (48, 50_001, "bf16"), (5, 70_003, "f32"), (33, 20_011, "bf16"),
                                       (64, 2_048, "bf16"), (2, 1_300, "f32")])
def test_several_steps_in_one_launch_equal_single_steps(rps_mod, oracle, n, d, dtype):
    """rps_step_n issues consecutive steps as one launch of the streamed kernel (fuse_steps): its teams go from step
    to step on their own tiles.  Bit for bit the result of one launch per step, across windows of masks, across
    t = 2^32, in shards, upwards only, with a ring longer than a step's tiles, and against the oracle's run."""
    w = wl.Workload("fused", n=n, d=d, dtype=dtype, p=0.15, gamma=0.05, sigma=0.1, seed=21 + n, steps=11)
    b = wl.make_targets(w)
    x0 = start(w, 6)
    every = (dict(), dict(mask_window=4), dict(traversal=1), dict(stages=8, consumer_warps=8, team_warps=2),
             dict(store_mode=2), dict(workers_per_lane=2, consumer_warps=3, team_warps=1))
    for t0 in (0, 27, (1 << 32) - 5):
        single = run(rps_mod, w, b, x0, w.steps, t0=t0, kernel=4, fuse_steps=1)
        for opts in (every if t0 == 27 else every[:2]):
            ref = single if "traversal" not in opts else run(rps_mod, w, b, x0, w.steps, t0=t0, kernel=4, fuse_steps=1,
                                                             traversal=1)
            got = run(rps_mod, w, b, x0, w.steps, t0=t0, kernel=4, fuse_steps=2, **opts)
            assert (got == ref).all(), (t0, opts, int((got != ref).sum()))
    want = x0.copy()
    oracle.run(want, b, dtype=dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=27, steps=w.steps)
    got = run(rps_mod, w, b, x0, w.steps, t0=27, kernel=4)
    assert rel_err(w, got, want) <= (BF16_TOL if dtype == "bf16" else RUN_TOL)
    # shards
    if d > 100_000:
        pieces = [(0, 64_000), (64_000, 36_032), (100_032, d - 100_032)]
        parts = [run(rps_mod, w, b, x0, w.steps, t0=27, shard=piece, kernel=4) for piece in pieces]
        assert (np.concatenate(parts, axis=1) == got).all()


def test_fused_launches_are_counted_and_tracked_steps_stay_single(rps_mod):
    w = wl.Workload("fused", n=64, d=65_536, dtype="bf16", p=0.1, gamma=0.05, sigma=0.1, seed=3, steps=40)
    b = wl.make_targets(w)
    r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype="bf16", sigma=w.sigma, kernel=4)
    r.set_targets(b)
    before = r.launch_count()
    r.step_n(40)  # masks of 32 steps, 32 steps in one launch; masks again, 8 steps in one launch
    assert r.launch_count() - before == 4 and r.get_step() == 40
    r.track(3)
    before = r.launch_count()
    r.step_n(5)   # three tracked steps singly, then two in one launch (no new masks: steps 40..44 of the window 32..63)
    assert r.launch_count() - before == 4 and r.read_trace().shape == (3, 2)
    r.close()


@pytest.mark.parametrize("dtype,n,d,extra,kernel", [
    ("f32", 12, 70_001, {}, 4), ("f32", 16, 70_001, {}, 2), ("f32", 6, 100_003, dict(average_gradients=True), 4),
    ("f32", 2, 300_007, {}, 4),
    ("bf16", 24, 70_001, {}, 4), ("bf16", 16, 100_003, {}, 3), ("bf16", 4, 200_003, {}, 4), ("bf16", 64, 50_001, {}, 4),
    ("bf16", 12, 100_003, dict(average_gradients=True), 4), ("bf16", 28, 70_001, dict(average_gradients=True), 3),
    ("bf16", 3, 300_007, dict(average_gradients=True), 4), ("bf16", 64, 50_001, dict(average_gradients=True), 3),
])
def test_the_librarys_own_choice_of_kernel(rps_mod, dtype, n, d, extra, kernel):
    """The lane groups of the staged and ring kernels are padded to a power of two of workers, the streamed kernel's
    time is proportional to n: left to itself the library takes the streamed kernel between two powers of two (and
    for bf16 replicas of fewer than 8 or more than 32 workers), the others where their groups are full.  Seen in
    the bits: the summation order differs between the forms."""
    w = wl.Workload("choice", n=n, d=d, dtype=dtype, p=0.2, gamma=0.05, sigma=0.1, seed=40 + n, steps=3)
    b = wl.make_targets(w)
    x0 = start(w, 8)
    own = run(rps_mod, w, b, x0, w.steps, strict_padding=kernel == 4, **extra)  # (only the streamed kernel never writes padding)
    assert (own == run(rps_mod, w, b, x0, w.steps, strict_padding=False, kernel=kernel, **extra)).all()
    if n > 4:  # with up to 4 workers every form adds them up in the same order
        others = [k for k in (2, 3, 4) if k != kernel and not (k == 3 and dtype == "f32")]
        assert any((own != run(rps_mod, w, b, x0, w.steps, strict_padding=False, kernel=k, **extra)).any() for k in others)
