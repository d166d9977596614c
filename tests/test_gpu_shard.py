"""Column shards: handles that each hold a range of the model's columns, stepped independently, must produce
bit for bit what one handle holding the whole model produces (same lane shape), because columns never
interact and masks and noise are pure functions of (seed, t, block, worker, column).  The whole-model
handle is itself checked against the oracle by the parity tests; here the oracle checks one sharded run too."""
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


def run_sharded(rps_mod, w, b, x0, world, **kw):
    parts = []
    traces = []
    for rank in range(world):
        begin, cols = rps_mod.shard_columns(w.d, world, rank)
        if cols == 0:
            continue
        r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, dtype=w.dtype, sigma=w.sigma, shard_begin=begin,
                        shard_cols=cols, **kw)
        r.set_targets(np.ascontiguousarray(b[:, begin:begin + cols]))
        r.write(np.ascontiguousarray(x0[:, begin:begin + cols]))
        r.track(w.steps)
        r.step_n(w.steps)
        parts.append(r.read())
        traces.append(r.read_trace())
        r.close()
    return np.concatenate(parts, axis=1), np.sum(traces, axis=0)


@pytest.mark.parametrize("n,d,dtype", [(8, 300_011, "f32"), (5, 70_001, "f32"), (32, 50_005, "f32"), (64, 40_000, "bf16"),
                                       (3, 1_000, "f32")])
@pytest.mark.parametrize("kernel", [1, 2])
def test_shards_reproduce_the_whole_model_bit_for_bit(rps_mod, n, d, dtype, kernel):
    w = wl.Workload("shard", n=n, d=d, dtype=dtype, p=0.15, gamma=0.1, sigma=0.1, seed=31 + n, steps=4, hetero=True)
    b = wl.make_targets(w)
    rng = np.random.default_rng(5)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    if dtype == "bf16":
        x0 = wl.f32_to_bf16_bits(x0)
    whole = rps_mod.RPS(n, d, w.p, w.gamma, w.seed, dtype=dtype, sigma=w.sigma, kernel=kernel, workers_per_lane=4)
    whole.set_targets(b)
    whole.write(x0)
    whole.track(w.steps)
    whole.step_n(w.steps)
    want = whole.read()
    want_trace = whole.read_trace()
    whole.close()
    bits = np.uint16 if dtype == "bf16" else np.uint32
    for world in (2, 3, 7):
        got, trace = run_sharded(rps_mod, w, b, x0, world, kernel=kernel, workers_per_lane=4)
        assert got.shape == want.shape
        assert (got.view(bits) == want.view(bits)).all(), world
        # both diagnostics are sums over columns: the shards' traces add up to the whole model's
        assert np.allclose(trace, want_trace, rtol=1e-9, atol=1e-12)


def test_a_sharded_run_matches_the_oracle(rps_mod, oracle):
    """Library defaults on each shard (small shards take the direct kernel, large ones the staged one)."""
    w = wl.WORKLOADS["cfg2"].scaled(d=400_010, steps=10)
    b = wl.make_targets(w)
    x0 = wl.make_initial(w)
    want = x0.copy()
    oracle.run(want, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
    got, _ = run_sharded(rps_mod, w, b, x0, 5)
    err = np.abs(got.astype(np.float64) - want.astype(np.float64)) / (1.0 + np.abs(want.astype(np.float64)))
    assert err.max() <= 1e-5, err.max()
