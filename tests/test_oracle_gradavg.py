"""Pins for the oracle's gradient-averaging comparison (Section 5, "Comparison with Gradient
Averaging"): the global view with the same matrix W, closed forms, and the paper's point that a
drop leaves an error between replicas that never decays.  CPU only."""
import math

import numpy as np
import pytest

from paper_1810_07766_b200 import workloads as wl
from test_oracle_step import mask_words, patterns, w_matrix


@pytest.mark.parametrize("n", [2, 3])
def test_gradavg_is_x_plus_update_times_w(oracle, n):
    """With U = V - X the updates -gamma*g, one step is X + U W for the W of Eq. 3: a receiver applies
    the average update over the arrived copies, everybody else its own."""
    rng = np.random.default_rng(n)
    d = 2 * n + 1
    block = oracle.block_size(n, d)
    gamma = 0.25
    b = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    x64 = x0.astype(np.float64)
    u = -float(np.float32(gamma)) * (x64 - b)
    pats = [(up, dn) for up, dn, _ in patterns(n, 0, 0.5)] + [([0] * n, [1] * n)]
    for a in range(len(pats)):
        for c in range(0, len(pats), 3):
            per_block = [pats[a] if j % 2 == 0 else pats[c] for j in range(n)]
            per_block = [(list(np.roll(up, j)), list(np.roll(dn, j))) for j, (up, dn) in enumerate(per_block)]
            up, down = mask_words(n, per_block)
            x = x0.copy()
            oracle.step(x, b, dtype="f32", gamma=gamma, sigma=0.0, p=0.5, seed=1, t=0, forced_up=up, forced_down=down,
                        average_gradients=True)
            want = np.empty((n, d))
            for j in range(n):
                cols = slice(j * block, min((j + 1) * block, d))
                want[:, cols] = x64[:, cols] + (u[:, cols].T @ w_matrix(n, *per_block[j])).T
            assert np.abs(x - want).max() <= 1e-6


def test_gradavg_without_drops_moves_every_replica_by_the_mean_gradient(oracle):
    n, d = 5, 31
    rng = np.random.default_rng(0)
    b = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    x = x0.copy()
    oracle.step(x, b, dtype="f32", gamma=0.1, sigma=0.0, p=0.0, seed=3, t=0, average_gradients=True)
    g = x0.astype(np.float64) - b
    assert np.abs(x - (x0 - float(np.float32(0.1)) * g.mean(axis=0))).max() <= 1e-6
    # from a common model the lossless baseline is the same as model averaging (Section 5)
    common = np.repeat(x0[:1], n, axis=0)
    a, m = common.copy(), common.copy()
    oracle.step(a, b, dtype="f32", gamma=0.1, sigma=0.3, p=0.0, seed=3, t=1, average_gradients=True)
    oracle.step(m, b, dtype="f32", gamma=0.1, sigma=0.3, p=0.0, seed=3, t=1)
    assert np.abs(a.astype(np.float64) - m).max() <= 1e-6


def test_gradavg_with_everything_lost_is_local_sgd(oracle):
    n, d = 4, 17
    rng = np.random.default_rng(1)
    b = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    a, m = x0.copy(), x0.copy()
    oracle.step(a, b, dtype="f32", gamma=0.2, sigma=0.1, p=1.0, seed=5, t=2, average_gradients=True)
    oracle.step(m, b, dtype="f32", gamma=0.2, sigma=0.1, p=1.0, seed=5, t=2)
    assert np.abs(a.astype(np.float64) - m).max() <= 1e-6


def test_dropped_messages_leave_an_error_that_never_decays(oracle):
    """The paper's reason for model averaging: under gradient averaging a replica that misses an average
    keeps the difference for ever (replicas that all receive the same average move in parallel), whereas
    model averaging wipes differences out at every delivery."""
    w = wl.Workload("cmp", n=8, d=512, dtype="f32", p=0.05, gamma=0.05, sigma=0.1, seed=11, steps=400)
    b = np.repeat(wl.make_targets(w)[:1], w.n, axis=0)          # one common optimum: any spread is the method's
    spread = {}
    for grad in (False, True):
        x = wl.make_initial(w)
        seen = []
        for t0 in range(0, w.steps, 100):
            oracle.run(x, b, dtype="f32", gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=t0, steps=100,
                       average_gradients=grad)
            seen.append(oracle.diag(x, b, dtype="f32")[1] / (w.n * w.d))
        spread[grad] = seen
    assert spread[True][-1] > 5 * spread[False][-1]
    # a step in which everything is delivered: model averaging ends in consensus, gradient averaging keeps its spread
    x_m, x_g = (np.random.default_rng(2).standard_normal(b.shape).astype(np.float32) for _ in range(2))
    before = oracle.diag(x_g, b, dtype="f32")[1]
    oracle.step(x_m, b, dtype="f32", gamma=0.05, sigma=0.0, p=0.0, seed=1, t=0)
    oracle.step(x_g, b, dtype="f32", gamma=0.05, sigma=0.0, p=0.0, seed=1, t=0, average_gradients=True)
    assert oracle.diag(x_m, b, dtype="f32")[1] == 0.0
    assert oracle.diag(x_g, b, dtype="f32")[1] == pytest.approx(before, rel=1e-5)
