"""Pins for the oracle's Monte-Carlo estimate of alpha_1 and alpha_2 (Eqs. 4 and 5, plotted in
Figures 2 and 3): the exact values from every drop pattern on tiny n, the two ends p = 0 and
p = 1, the orders the paper states, and a second route to the per-sample value."""
import math

import numpy as np
import pytest

from test_oracle_step import patterns, w_matrix


def exact_alphas(n, p):
    """alpha_1, alpha_2 by summing over every drop pattern and every server (drawn uniformly)."""
    a_n = np.full((n, n), 1.0 / n)
    eww = np.zeros((n, n))
    ewaw = np.zeros((n, n))
    for server in range(n):
        for up, down, prob in patterns(n, server, p):
            w = w_matrix(n, up, down)
            eww += prob / n * w @ w.T
            ewaw += prob / n * w @ a_n @ w.T
    return eww[0, 0] - eww[0, 1], ewaw[0, 0] - ewaw[0, 1]


@pytest.mark.parametrize("n,p,assign", [(2, 0.3, 0), (3, 0.2, 0), (3, 0.2, 1), (4, 0.4, 1), (5, 0.1, 0)])
def test_estimate_converges_to_the_exact_alphas(oracle, n, p, assign):
    a1, a2 = exact_alphas(n, p)
    steps = 40_000
    got1, got2 = oracle.alpha_mc(n, p, 2024 + n, 0, steps, assign=assign)
    # a sample lies in [0, 1]: its standard deviation is at most 1/2, and there are n * steps of them
    # (independent across steps); 5 sigma
    bound = 5 * 0.5 / math.sqrt(steps)
    assert abs(got1 - a1) < bound, (got1, a1)
    assert abs(got2 - a2) < bound, (got2, a2)
    assert 0 < got2 < got1 < 1


def test_ends_of_the_drop_rate(oracle):
    for n in (2, 5, 16, 64):
        # nothing lost: W = A_n, so W W^T = W A_n W^T = A_n and both constants vanish
        a1, a2 = oracle.alpha_mc(n, 0.0, 1, 0, 8)
        assert abs(a1) < 1e-12 and abs(a2) < 1e-12
        # everything lost (the server still has its own copy): W = I, so W W^T = I and W A_n W^T = A_n
        a1, a2 = oracle.alpha_mc(n, 1.0, 1, 0, 8)
        assert abs(a1 - 1.0) < 1e-12 and abs(a2) < 1e-12
        # without self-delivery the same ends hold: W = A_n, and W = I when no average exists
        a1, a2 = oracle.alpha_mc(n, 1.0, 1, 0, 8, self_delivery=False)
        assert abs(a1 - 1.0) < 1e-12 and abs(a2) < 1e-12


def test_orders_stated_under_theorem_1(oracle):
    """alpha_2 = O(p (1 - p) / n) and beta = alpha_1 - alpha_2 = O(p): more workers shrink alpha_2 at a
    fixed drop rate, and beta stays of the order of p."""
    p = 0.1
    seen = []
    for n in (4, 8, 16, 32):
        a1, a2 = oracle.alpha_mc(n, p, 9, 0, 4000)
        seen.append(a2)
        assert a2 < 2.0 * p * (1 - p) / n * 4          # a generous constant; the trend is the point
        assert 0.5 * p < a1 - a2 < 2.0 * p
    assert all(later < earlier for earlier, later in zip(seen, seen[1:]))


def test_per_sample_value_by_counting(oracle):
    """A second route to one sample: with c arrivals (the set N), R receivers, and s_m the row sums of W,
    W W^T has trace R/c + n - R and total n, and W A_n W^T = s s^T / n with sum(s) = n."""
    n, p, seed = 6, 0.35, 5
    for t in range(50):
        up, down, cnt, _ = oracle.masks(n, p, seed, t)
        want1 = want2 = 0.0
        for j in range(n):
            u = [(int(up[j]) >> m) & 1 for m in range(n)]
            r = [(int(down[j]) >> m) & 1 for m in range(n)]
            c, big_r = int(cnt[j]), sum(r)
            trace1 = big_r / c + n - big_r
            s = [big_r * u[m] / c + (1 - r[m]) for m in range(n)]
            assert sum(s) == pytest.approx(n)
            trace2 = sum(v * v for v in s) / n
            want1 += trace1 / n - (n - trace1) / (n * (n - 1))
            want2 += trace2 / n - (n - trace2) / (n * (n - 1))
        got1, got2 = oracle.alpha_mc(n, p, seed, t, 1)
        assert got1 == pytest.approx(want1 / n, abs=1e-12)
        assert got2 == pytest.approx(want2 / n, abs=1e-12)
