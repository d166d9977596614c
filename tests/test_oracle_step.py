"""Pins for the oracle's step: the global view X_{t+1} = V_t W_t (Eq. 3), the exact
sums printed in the proofs of Lemmas 7 and 8, Eqs. 4 and 5, and closed forms.

The matrix W is built here from the paper's definition (independently of the
oracle's per-column code), checked against the paper's printed expressions by
exact enumeration of all drop patterns, and only then used to check the oracle.
None of these tests touches the CUDA library.
"""
import itertools
import math

import numpy as np
import pytest
import torch

from paper_1810_07766_b200 import workloads as wl


# ---------------------------------------------------------------- W of Eq. 3, by definition

def w_matrix(n, up_bits, down_bits):
    """[W]_{m,k}: weight of v^(m) in x_{t+1}^(k) for one block (Section 4.2).

    up_bits[m] = 1 iff worker m's copy reached the server, down_bits[k] = 1 iff
    worker k received the average.  A receiver's column is the uniform average
    over the arrived copies; everybody else keeps its own v (column e_k).
    """
    arrived = [m for m in range(n) if up_bits[m]]
    w = np.zeros((n, n))
    for k in range(n):
        if down_bits[k] and arrived:
            for m in arrived:
                w[m, k] = 1.0 / len(arrived)
        else:
            w[k, k] = 1.0
    return w


def patterns(n, server, p):
    """All drop patterns of one block with the server's own bits fixed to 1, with probabilities."""
    others = [i for i in range(n) if i != server]
    for ups in itertools.product((0, 1), repeat=n - 1):
        for downs in itertools.product((0, 1), repeat=n - 1):
            up = [1] * n
            down = [1] * n
            prob = 1.0
            for idx, i in enumerate(others):
                up[i], down[i] = ups[idx], downs[idx]
                prob *= (1 - p) if ups[idx] else p
                prob *= (1 - p) if downs[idx] else p
            yield up, down, prob


def comb(a, b):
    return math.comb(a, b)


@pytest.mark.parametrize("n,p", [(2, 0.3), (3, 0.1), (4, 0.25), (5, 0.6)])
def test_w_matches_the_exact_sums_in_the_proofs(n, p):
    q = 1 - p
    # Case 1 of Lemma 7: node 1 serves the block (event A).
    e_w11_sq = e_row_sq = e_row_sum_sq = total = 0.0
    for up, down, prob in patterns(n, 0, p):
        w = w_matrix(n, up, down)
        total += prob
        e_w11_sq += prob * w[0, 0] ** 2
        e_row_sq += prob * (w[0] ** 2).sum()
        e_row_sum_sq += prob * w[0].sum() ** 2
    assert total == pytest.approx(1.0, abs=1e-12)
    paper_w11_sq = sum(comb(n - 1, m) * q ** m * p ** (n - 1 - m) / (m + 1) ** 2 for m in range(n))
    assert e_w11_sq == pytest.approx(paper_w11_sq, rel=1e-12)
    assert e_row_sq == pytest.approx(paper_w11_sq * (1 + (n - 1) * q), rel=1e-12)            # Eq. (21)
    assert e_row_sum_sq == pytest.approx(
        paper_w11_sq * ((1 + (n - 1) * q) ** 2 + (n - 1) * p * q), rel=1e-12)                # Lemma 8, Case 1

    # Cases 2 and 3: node n serves the block; C = node 1 did not receive the average.
    acc = {0: dict(pr=0.0, w1n=0.0, w1n_sq=0.0, row_sq=0.0, row_sum_sq=0.0),
           1: dict(pr=0.0, w11_sq=0.0, row_sq=0.0, row_sum_sq=0.0)}
    for up, down, prob in patterns(n, n - 1, p):
        w = w_matrix(n, up, down)
        if down[0] == 0:
            a = acc[0]
            a["pr"] += prob
            a["w1n"] += prob * w[0, n - 1]
            a["w1n_sq"] += prob * w[0, n - 1] ** 2
            a["row_sq"] += prob * (w[0] ** 2).sum()
            a["row_sum_sq"] += prob * w[0].sum() ** 2
        else:
            a = acc[1]
            a["pr"] += prob
            a["w11_sq"] += prob * w[0, 0] ** 2
            a["row_sq"] += prob * (w[0] ** 2).sum()
            a["row_sum_sq"] += prob * w[0].sum() ** 2
    assert acc[0]["pr"] == pytest.approx(p) and acc[1]["pr"] == pytest.approx(q)              # E[B] = 1 - p
    paper_w1n = sum(comb(n - 2, m) * q ** (m + 1) * p ** (n - 2 - m) / (m + 2) for m in range(n - 1))
    paper_w1n_sq = sum(comb(n - 2, m) * q ** (m + 1) * p ** (n - 2 - m) / (m + 2) ** 2 for m in range(n - 1))
    assert acc[0]["w1n"] / p == pytest.approx(paper_w1n, rel=1e-12)
    assert acc[0]["w1n_sq"] / p == pytest.approx(paper_w1n_sq, rel=1e-12)
    assert acc[0]["row_sq"] / p == pytest.approx(1 + paper_w1n_sq * (1 + (n - 2) * q), rel=1e-12)
    e_b = (n - 2) * q + 1
    e_b_sq = 1 + 2 * (n - 2) * q + (n - 2) ** 2 * q ** 2 + (n - 2) * p * q
    assert acc[0]["row_sum_sq"] / p == pytest.approx(1 + 2 * paper_w1n * e_b + paper_w1n_sq * e_b_sq, rel=1e-12)
    assert acc[1]["w11_sq"] / q == pytest.approx(paper_w1n_sq, rel=1e-12)                     # Case 3
    assert acc[1]["row_sq"] / q == pytest.approx(paper_w1n_sq * (2 + (n - 2) * q), rel=1e-12)
    assert acc[1]["row_sum_sq"] / q == pytest.approx(
        paper_w1n_sq * (((n - 2) * q + 2) ** 2 + (n - 2) * p * q), rel=1e-12)
    # the closed upper bound T3 / n of Lemma 8
    if n >= 3:
        t3 = n / (n - 1) * (1 - p ** (n - 1) - q ** (n - 1)) + q ** (n - 1)
        assert paper_w1n <= t3 / n + 1e-12


@pytest.mark.parametrize("n,p", [(3, 0.2), (4, 0.4)])
def test_expected_w_has_the_structure_of_eqs_4_and_5(n, p):
    """With the server drawn uniformly (Algorithm 1), E[W], E[W W^T], E[W A_n W^T] are
    alpha*I + (1-alpha)*A_n, E[W] A_n = A_n, and 0 < alpha_2 < alpha_1 < 1."""
    a_n = np.full((n, n), 1.0 / n)
    ew = np.zeros((n, n))
    eww = np.zeros((n, n))
    ewaw = np.zeros((n, n))
    for server in range(n):
        for up, down, prob in patterns(n, server, p):
            w = w_matrix(n, up, down)
            ew += prob / n * w
            eww += prob / n * w @ w.T
            ewaw += prob / n * w @ a_n @ w.T

    def alpha_of(m):
        off = m[0, 1]
        diag = m[0, 0]
        assert np.allclose(m - np.diag(np.diag(m)), off * (1 - np.eye(n)), atol=1e-12)
        assert np.allclose(np.diag(m), diag, atol=1e-12)
        alpha = diag - off
        assert np.allclose(m, alpha * np.eye(n) + (1 - alpha) * a_n, atol=1e-12)
        return alpha

    alpha_of(ew)
    assert np.allclose(ew @ a_n, a_n, atol=1e-12)
    alpha1 = alpha_of(eww)
    alpha2 = alpha_of(ewaw)
    assert 0 < alpha2 < alpha1 < 1
    q = 1 - p
    t1 = 2 * (1 - p ** (n + 1) - (n + 1) * q * p ** n - (n + 1) * n * q * q * p ** (n - 1) / 2 - q ** (n + 1)) / (
        n * (n + 1) * q * q)
    t2 = (1 - p ** n - n * q * p ** (n - 1) - q ** n) / ((n - 1) * q)
    assert alpha1 <= (n * p + q ** n + n * t1 + n * t2 - 1) / (n - 1) + 1e-12                # Lemma 7's bound


def test_w_is_column_stochastic_not_doubly_stochastic():
    n = 4
    seen_non_doubly = False
    for up, down, _ in patterns(n, 1, 0.5):
        w = w_matrix(n, up, down)
        assert np.allclose(w.sum(axis=0), 1.0)
        seen_non_doubly |= not np.allclose(w.sum(axis=1), 1.0)
    assert seen_non_doubly


# ---------------------------------------------------------------- the oracle against V W

def mask_words(n, per_block):
    up = np.zeros(n, dtype=np.uint64)
    down = np.zeros(n, dtype=np.uint64)
    for j, (u, dn) in enumerate(per_block):
        up[j] = sum(1 << i for i in range(n) if u[i])
        down[j] = sum(1 << i for i in range(n) if dn[i])
    return up, down


@pytest.mark.parametrize("n", [2, 3])
def test_step_equals_v_times_w_for_every_drop_pattern(oracle, n):
    rng = np.random.default_rng(100 + n)
    d = 2 * n + 1                       # ragged: block size ceil(d/n) = 3, last block short
    block = oracle.block_size(n, d)
    assert block == -(-d // n)
    gamma = 0.25
    b = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    v = x0.astype(np.float64) - float(np.float32(gamma)) * (x0.astype(np.float64) - b.astype(np.float64))
    all_patterns = [(u, dn) for u, dn, _ in patterns(n, 0, 0.5)]
    # also patterns in which the server's own bits are off (only reachable through forced masks)
    all_patterns += [([0] * n, [1] * n), ([1] + [0] * (n - 1), [0] * n)]
    for combo in itertools.product(range(len(all_patterns)), repeat=2):
        per_block = [all_patterns[combo[j % 2]] for j in range(n)]
        # rotate so that block j's "server" pattern is not always worker 0
        per_block = [(list(np.roll(u, j)), list(np.roll(dn, j))) for j, (u, dn) in enumerate(per_block)]
        up, down = mask_words(n, per_block)
        x = x0.copy()
        oracle.step(x, b, dtype="f32", gamma=gamma, sigma=0.0, p=0.5, seed=1, t=0, forced_up=up, forced_down=down)
        want = np.empty((n, d))
        for j in range(n):
            cols = slice(j * block, min((j + 1) * block, d))
            w = w_matrix(n, *per_block[j])
            want[:, cols] = (v[:, cols].T @ w).T        # X^(j) = V^(j) W^(j), workers as columns
        assert np.abs(x - want).max() <= 1e-6


def test_two_worker_outcomes_by_hand(oracle):
    """n = 2, block 0 served by worker 0: the four outcomes of (up, down) for worker 1."""
    b = np.array([[2.0, 0.0], [6.0, 0.0]], dtype=np.float32)
    gamma = 0.5
    v0, v1 = 1.0, 3.0                    # x = 0 -> v = gamma * b
    cases = {(1, 1): (2.0, 2.0), (1, 0): (2.0, v1), (0, 1): (v0, v0), (0, 0): (v0, v1)}
    for (u1, d1), (want0, want1) in cases.items():
        x = np.zeros((2, 2), dtype=np.float32)
        up = np.array([1 | (u1 << 1), 3], dtype=np.uint64)
        down = np.array([1 | (d1 << 1), 3], dtype=np.uint64)
        oracle.step(x, b, dtype="f32", gamma=gamma, sigma=0.0, p=0.0, seed=0, t=0, forced_up=up, forced_down=down)
        assert (x[0, 0], x[1, 0]) == (want0, want1)


def test_sampled_step_equals_v_times_w_of_its_own_masks(oracle):
    n, d = 5, 23
    rng = np.random.default_rng(5)
    b = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    block = oracle.block_size(n, d)
    for assign in (oracle.ASSIGN_FIXED, oracle.ASSIGN_PERM):
        for t in range(10):
            up, down, cnt, _ = oracle.masks(n, 0.4, 8, t, assign=assign)
            x = x0.copy()
            oracle.step(x, b, dtype="f32", gamma=0.1, sigma=0.0, p=0.4, seed=8, t=t, assign=assign)
            v = x0.astype(np.float64) - float(np.float32(0.1)) * (x0.astype(np.float64) - b)
            for j in range(n):
                cols = slice(j * block, min((j + 1) * block, d))
                w = w_matrix(n, [(int(up[j]) >> i) & 1 for i in range(n)], [(int(down[j]) >> i) & 1 for i in range(n)])
                assert np.abs(x[:, cols] - (v[:, cols].T @ w).T).max() <= 1e-6


def test_noise_enters_the_gradient_with_sigma_and_gamma(oracle):
    n, d = 3, 10
    b = np.zeros((n, d), dtype=np.float32)
    x = np.zeros((n, d), dtype=np.float32)
    gamma, sigma = 0.5, 0.25
    oracle.step(x, b, dtype="f32", gamma=gamma, sigma=sigma, p=1.0, seed=6, t=4)   # p = 1: x_{t+1} = v
    for i in range(n):
        for c in range(d):
            assert x[i, c] == np.float32(-gamma * sigma * oracle.noise(6, 4, i, c))


# ---------------------------------------------------------------- closed forms

def test_p0_is_the_exact_mean_of_local_sgd(oracle):
    w = wl.WORKLOADS["cfg1"].scaled(d=1000)
    b = wl.make_targets(w)
    x = wl.make_initial(w)
    bbar = b.astype(np.float64).mean(axis=0)
    g = float(np.float32(w.gamma))
    for t in range(1, 31):
        oracle.step(x, b, dtype="f32", gamma=w.gamma, sigma=0.0, p=0.0, seed=w.seed, t=t - 1)
        assert (x == x[0]).all()                                         # consistent replicas
        assert np.abs(x[0] - (1 - (1 - g) ** t) * bbar).max() <= 1e-6    # x_t = (1-(1-gamma)^t) mean(b)
    # one noisy step from a non-trivial state: every replica equals mean_k v^(k)
    x0 = np.random.default_rng(0).standard_normal(b.shape).astype(np.float32)
    x = x0.copy()
    oracle.step(x, b, dtype="f32", gamma=w.gamma, sigma=w.sigma, p=0.0, seed=3, t=9)
    xi = np.array([[oracle.noise(3, 9, i, c) for c in range(w.d)] for i in range(w.n)])
    v = x0 - g * ((x0.astype(np.float64) - b) + float(np.float32(w.sigma)) * xi)
    assert np.abs(x - v.mean(axis=0)).max() <= 1e-6


def test_p1_is_pure_local_sgd(oracle):
    w = wl.WORKLOADS["cfg1"].scaled(d=1000)
    b = wl.make_targets(w)
    x = wl.make_initial(w)
    g = float(np.float32(w.gamma))
    for t in range(1, 31):
        oracle.step(x, b, dtype="f32", gamma=w.gamma, sigma=0.0, p=1.0, seed=w.seed, t=t - 1)
        assert np.abs(x - (1 - (1 - g) ** t) * b.astype(np.float64)).max() <= 1e-6


def test_outputs_are_convex_combinations_and_receivers_agree(oracle):
    n, d = 8, 203
    rng = np.random.default_rng(2)
    b = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    block = oracle.block_size(n, d)
    for t in range(5):
        x = x0.copy()
        oracle.step(x, b, dtype="f32", gamma=0.1, sigma=0.0, p=0.3, seed=2, t=t)
        v = (x0.astype(np.float64) - float(np.float32(0.1)) * (x0.astype(np.float64) - b))
        assert (x <= v.max(axis=0) + 1e-6).all() and (x >= v.min(axis=0) - 1e-6).all()
        _, down, _, _ = oracle.masks(n, 0.3, 2, t)
        for j in range(n):
            rows = [i for i in range(n) if (int(down[j]) >> i) & 1]
            cols = slice(j * block, min((j + 1) * block, d))
            assert (x[rows, cols] == x[rows[0], cols]).all()


def test_expected_mean_moves_by_the_mean_sgd_step(oracle):
    """Lemma 4: E[xbar_{t+1}] = vbar_t when the servers are drawn uniformly (Monte Carlo
    over the oracle's own sampled masks and permutations)."""
    n, d, p, trials = 4, 4, 0.3, 20000
    rng = np.random.default_rng(3)
    b = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    v = x0.astype(np.float64) - float(np.float32(0.2)) * (x0.astype(np.float64) - b)
    means = np.empty((trials, d))
    for t in range(trials):
        x = x0.copy()
        oracle.step(x, b, dtype="f32", gamma=0.2, sigma=0.0, p=p, seed=77, t=t, assign=oracle.ASSIGN_PERM)
        means[t] = x.mean(axis=0)
    err = means.mean(axis=0) - v.mean(axis=0)
    se = means.std(axis=0) / math.sqrt(trials)
    assert (np.abs(err) < 4.5 * se + 1e-7).all()


def test_quadratic_converges_to_a_ball_around_the_optimum(oracle):
    """Constant step size converges to a ball (Section 5 discussion); for the quadratic the
    centre is mean_i b_i and the radius is set by gamma, sigma, n and p."""
    w = wl.WORKLOADS["cfg1"].scaled(d=2048)
    b = wl.make_targets(w)
    x = wl.make_initial(w)
    oracle.run(x, b, dtype="f32", gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t0=0, steps=w.steps)
    dist2, cons = oracle.diag(x, b, dtype="f32")
    rms = math.sqrt(dist2 / w.d)
    assert rms < 0.06                        # started at distance ~ 0.5
    start = math.sqrt((b.astype(np.float64).mean(axis=0) ** 2).mean())
    assert rms < 0.15 * start
    # the noiseless, lossless run reaches the optimum itself
    x = wl.make_initial(w)
    oracle.run(x, b, dtype="f32", gamma=w.gamma, sigma=0.0, p=0.0, seed=w.seed, t0=0, steps=200)
    dist2, cons = oracle.diag(x, b, dtype="f32")
    assert math.sqrt(dist2 / w.d) < 1e-6 and cons == 0.0


def test_diag_against_numpy(oracle):
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 77)).astype(np.float32)
    b = rng.standard_normal((5, 77)).astype(np.float32)
    dist2, cons = oracle.diag(x, b, dtype="f32")
    x64, b64 = x.astype(np.float64), b.astype(np.float64)
    assert dist2 == pytest.approx(((x64.mean(0) - b64.mean(0)) ** 2).sum(), rel=1e-12)
    assert cons == pytest.approx(((x64 - x64.mean(0)) ** 2).sum(), rel=1e-12)


# ---------------------------------------------------------------- partition, columns, bf16

@pytest.mark.parametrize("n,d", [(4, 65536), (8, 11_173_962), (16, 25_557_032), (32, 4_000_037), (7, 3), (5, 5)])
def test_partition(oracle, n, d):
    blk = oracle.block_size(n, d)
    assert blk * n >= d and (blk - 1) * n < d


def test_step_columns_matches_full_step(oracle):
    w = wl.WORKLOADS["cfg4"].scaled(d=4001)
    b = wl.make_targets(w)
    rng = np.random.default_rng(0)
    x0 = rng.standard_normal(b.shape).astype(np.float32)
    full = x0.copy()
    oracle.step(full, b, dtype="f32", gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=5)
    cols = np.array([0, 1, 124, 125, 126, 2000, 3999, 4000], dtype=np.int64)
    xc = np.ascontiguousarray(x0[:, cols])
    bc = np.ascontiguousarray(b[:, cols])
    oracle.step_columns(w.d, cols, xc, bc, dtype="f32", gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=5)
    assert (xc == full[:, cols]).all()


def test_bf16_rounding_against_library_conversion(oracle):
    rng = np.random.default_rng(0)
    vals = np.concatenate([rng.standard_normal(5000).astype(np.float32) * 3,
                           (rng.standard_normal(2000) * 1e-3).astype(np.float32),
                           np.array([0.0, -0.0, 1.0, -1.0, 1.00390625, 1.01171875, 0.99609375, 3.0e-39, 65280.0],
                                    dtype=np.float32)])
    want = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.double_to_bf16(float(v)) for v in vals], dtype=np.uint16)
    assert (got == want).all()
    assert (wl.f32_to_bf16_bits(vals) == want).all()
    # ties to even, and a value only a double can tell from a tie
    assert oracle.double_to_bf16(1.00390625) == 0x3F80          # 1 + 2^-8: tie, even mantissa below
    assert oracle.double_to_bf16(1.01171875) == 0x3F82          # 1 + 3*2^-8: tie, even mantissa above
    assert oracle.double_to_bf16(1.00390625 + 2.0 ** -40) == 0x3F81
    for bits in (0x0000, 0x3F80, 0xBF80, 0x4049, 0x0001, 0x7F7F):
        assert oracle.double_to_bf16(oracle.bf16_to_double(bits)) == bits


def test_bf16_step_rounds_once_from_double(oracle):
    w = wl.WORKLOADS["cfg5"].scaled(d=512)
    b = wl.make_targets(w)
    x = wl.make_initial(w)
    x32 = np.zeros(b.shape, dtype=np.float32)
    b32 = wl.bf16_bits_to_f32(b)
    oracle.step(x, b, dtype="bf16", gamma=w.gamma, sigma=0.0, p=0.0, seed=w.seed, t=0)
    mean_v = (float(np.float32(w.gamma)) * b32.astype(np.float64)).mean(axis=0)
    want = np.array([oracle.double_to_bf16(float(v)) for v in mean_v], dtype=np.uint16)
    assert (x == want).all()
    del x32
