"""rps_estimate_alpha against the oracle's Monte-Carlo estimate over the same steps: the masks are
bit-exact, so the two average the same samples and may differ only by the order of fp64 additions
(the oracle multiplies the W matrices out; the device counts arrivals and receivers)."""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rps_mod():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_1810_07766_b200 import binding, build

    build.build()
    binding.load_library()
    return binding


@pytest.mark.parametrize("n", [2, 3, 8, 16, 33, 64])
def test_alpha_matches_the_oracle_sample_for_sample(rps_mod, oracle, n):
    for p, self_delivery, assign, window in ((0.1, True, 0, 32), (0.3, True, 1, 7), (0.05, False, 0, 256),
                                             (0.0, True, 0, 32), (1.0, True, 1, 32), (1.0, False, 0, 32)):
        seed = 0xA1FA0000 + n
        r = rps_mod.RPS(n, 4096, p, 0.1, seed, self_delivery=self_delivery, assign=assign, mask_window=window)
        for t0, steps in ((0, 300), ((1 << 32) - 5, 40), (17, 1)):
            got = r.estimate_alpha(t0, steps)
            want = oracle.alpha_mc(n, p, seed, t0, steps, self_delivery=self_delivery, assign=assign)
            assert got[0] == pytest.approx(want[0], abs=1e-12), (p, self_delivery, assign, t0)
            assert got[1] == pytest.approx(want[1], abs=1e-12), (p, self_delivery, assign, t0)
        r.close()


def test_alpha_leaves_the_run_alone(rps_mod, oracle):
    """Estimating in the middle of a run disturbs neither the replicas nor the step counter."""
    import numpy as np

    from paper_1810_07766_b200 import workloads as wl

    w = wl.Workload("mid", n=8, d=50_001, dtype="f32", p=0.2, gamma=0.1, sigma=0.1, seed=21, steps=6)
    b = wl.make_targets(w)
    out = []
    for interrupt in (False, True):
        r = rps_mod.RPS(w.n, w.d, w.p, w.gamma, w.seed, sigma=w.sigma)
        r.set_targets(b)
        r.step_n(3)
        if interrupt:
            a1, a2 = r.estimate_alpha(1000, 100)
            assert 0 < a2 < a1 < 1
            assert r.get_step() == 3
        r.step_n(3)
        out.append(r.read().view(np.uint32))
        r.close()
    assert (out[0] == out[1]).all()


def test_alpha_needs_two_workers(rps_mod):
    r = rps_mod.RPS(1, 1024, 0.1, 0.1, 1)
    with pytest.raises(rps_mod.RPSError):
        r.estimate_alpha(0, 10)
    r.close()
    r = rps_mod.RPS(4, 1024, 0.1, 0.1, 1)
    with pytest.raises(rps_mod.RPSError):
        r.estimate_alpha(0, 0)
    r.close()
