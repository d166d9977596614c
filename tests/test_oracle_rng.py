"""Pins for the oracle's random streams: Philox, drop masks, server draw, noise.

None of these tests touches the CUDA library.
"""
import math
import os

import numpy as np
import pytest
from scipy import stats

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def read_kat():
    rows = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(tok, 16) for tok in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers(oracle):
    rows = read_kat()
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert list(oracle.philox4x32_10(ctr, key)) == want


def test_philox_counter_and_key_sensitivity(oracle):
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    seen = {base}
    for w in range(4):
        ctr = [1, 2, 3, 4]
        ctr[w] += 1
        seen.add(oracle.philox4x32_10(ctr, [5, 6]))
    seen.add(oracle.philox4x32_10([1, 2, 3, 4], [6, 6]))
    seen.add(oracle.philox4x32_10([1, 2, 3, 4], [5, 7]))
    assert len(seen) == 7


# ----------------------------------------------------------------------------- masks

def bits(word, n):
    return [(int(word) >> i) & 1 for i in range(n)]


@pytest.mark.parametrize("n", [1, 2, 5, 64])
def test_masks_p0_everything_arrives(oracle, n):
    for sd in (True, False):
        up, down, cnt, server = oracle.masks(n, 0.0, 7, 3, self_delivery=sd)
        full = (1 << n) - 1
        assert all(int(u) == full for u in up) and all(int(v) == full for v in down)
        assert list(cnt) == [n] * n and list(server) == list(range(n))


@pytest.mark.parametrize("n", [1, 2, 5, 64])
def test_masks_p1_only_the_server_keeps_its_block(oracle, n):
    up, down, cnt, _ = oracle.masks(n, 1.0, 7, 3, self_delivery=True)
    assert [int(u) for u in up] == [1 << j for j in range(n)]
    assert [int(v) for v in down] == [1 << j for j in range(n)]
    assert list(cnt) == [1] * n
    up, down, cnt, _ = oracle.masks(n, 1.0, 7, 3, self_delivery=False)
    assert not up.any() and not down.any() and not cnt.any()


def test_masks_drop_rate_and_direction_independence(oracle):
    n, p = 64, 0.1
    lost_up = lost_down = both = total = 0
    for t in range(150):
        up, down, cnt, _ = oracle.masks(n, p, 11, t, self_delivery=False)
        for j in range(n):
            u, v = int(up[j]), int(down[j])
            assert cnt[j] == bin(u).count("1")
            if cnt[j] == 0:
                continue
            full = (1 << n) - 1
            lost_up += n - bin(u).count("1")
            lost_down += n - bin(v).count("1")
            both += bin(~u & ~v & full).count("1")
            total += n
    sd = math.sqrt(p * (1 - p) / total)
    assert abs(lost_up / total - p) < 4 * sd
    assert abs(lost_down / total - p) < 4 * sd
    # independent directions: P(both lost) = p^2
    sd2 = math.sqrt(p * p * (1 - p * p) / total)
    assert abs(both / total - p * p) < 4 * sd2


@pytest.mark.parametrize("n,p", [(8, 0.2), (16, 0.1)])
def test_receive_counts_follow_one_plus_binomial(oracle, n, p):
    """Proof of Lemma 7, Case 1: m of the other n-1 copies arrive with probability
    C(n-1,m)(1-p)^m p^(n-1-m); the server's own copy is always there."""
    obs = np.zeros(n + 1)
    steps = 4000
    for t in range(steps):
        _, _, cnt, _ = oracle.masks(n, p, 5, t)
        for c in cnt:
            obs[c] += 1
    assert obs[0] == 0
    expect = np.array([stats.binom.pmf(c - 1, n - 1, 1 - p) if c >= 1 else 0.0 for c in range(n + 1)]) * steps * n
    keep = expect > 5
    chi2 = ((obs[keep] - expect[keep]) ** 2 / expect[keep]).sum() + (obs[~keep].sum() - expect[~keep].sum()) ** 2 / max(
        expect[~keep].sum(), 1e-9)
    dof = keep.sum()
    assert chi2 < stats.chi2.ppf(0.9999, dof)


def test_counts_without_self_delivery_are_binomial_n(oracle):
    n, p, steps = 8, 0.3, 4000
    obs = np.zeros(n + 1)
    for t in range(steps):
        _, _, cnt, _ = oracle.masks(n, p, 9, t, self_delivery=False)
        for c in cnt:
            obs[c] += 1
    expect = stats.binom.pmf(np.arange(n + 1), n, 1 - p) * steps * n
    keep = expect > 5
    chi2 = ((obs[keep] - expect[keep]) ** 2 / expect[keep]).sum()
    assert chi2 < stats.chi2.ppf(0.9999, keep.sum())


def test_self_bits_forced_and_streams_unshifted(oracle):
    """Forcing the server's bits must not shift any other draw."""
    n, p = 16, 0.5
    for t in range(20):
        up1, down1, _, _ = oracle.masks(n, p, 3, t, self_delivery=True)
        up0, down0, cnt0, _ = oracle.masks(n, p, 3, t, self_delivery=False)
        for j in range(n):
            assert (int(up1[j]) >> j) & 1 and (int(down1[j]) >> j) & 1
            others = ((1 << n) - 1) & ~(1 << j)
            assert int(up1[j]) & others == int(up0[j]) & others
            if cnt0[j] > 0:
                assert int(down1[j]) & others == int(down0[j]) & others


def test_random_assignment_is_a_uniform_permutation(oracle):
    """Algorithm 1 draws the servers without replacement; P(worker 1 serves block 1) = 1/n."""
    n, steps = 6, 6000
    hits = np.zeros((n, n))
    for t in range(steps):
        up, down, _, server = oracle.masks(n, 0.5, 21, t, assign=oracle.ASSIGN_PERM)
        assert sorted(server) == list(range(n))
        for j in range(n):
            hits[j, server[j]] += 1
            assert (int(up[j]) >> int(server[j])) & 1 and (int(down[j]) >> int(server[j])) & 1
    expect = steps / n
    chi2 = ((hits - expect) ** 2 / expect).sum()
    assert chi2 < stats.chi2.ppf(0.9999, (n - 1) * (n - 1))
    # fixed assignment (Section 4.1): worker j serves block j
    assert list(oracle.masks(n, 0.5, 21, 0)[3]) == list(range(n))


def test_masks_depend_on_step_and_seed_not_on_d(oracle):
    a = oracle.masks(8, 0.5, 1, 0)
    assert any((a[0] != oracle.masks(8, 0.5, 1, 1)[0]))
    assert any((a[0] != oracle.masks(8, 0.5, 2, 0)[0]))
    b = oracle.masks(8, 0.5, 1, 0)
    assert all((a[k] == b[k]).all() for k in range(4))
    assert any((a[0] != oracle.masks(8, 0.5, 1, 1 << 32)[0]))  # high half of the step counts


# ----------------------------------------------------------------------------- noise

def noise_block(oracle, seed, t, workers, cols):
    return np.array([[oracle.noise(seed, t, i, c) for c in cols] for i in workers])


def test_noise_is_standard_normal(oracle):
    z = noise_block(oracle, 4, 17, range(8), range(0, 20000)).ravel()
    assert abs(z.mean()) < 4 / math.sqrt(z.size)
    assert abs(z.var() - 1.0) < 4 * math.sqrt(2.0 / z.size)
    assert abs(stats.kurtosis(z, fisher=False) - 3.0) < 4 * math.sqrt(24.0 / z.size)
    assert abs(stats.skew(z)) < 4 * math.sqrt(6.0 / z.size)
    assert stats.kstest(z, "norm").pvalue > 1e-4
    assert np.abs(z).max() <= math.sqrt(-2 * math.log(0.5 / 65536)) + 1e-12


def test_noise_columns_workers_steps_uncorrelated(oracle):
    a = noise_block(oracle, 4, 3, range(4), range(0, 8000))
    lim = 4.5 / math.sqrt(a.shape[1])
    for i in range(4):
        for k in range(i + 1, 4):
            assert abs(np.corrcoef(a[i], a[k])[0, 1]) < lim
    # neighbours inside one draw: the cosine/sine partners and the two pairs of a worker
    for lag in (1, 2, 3):
        assert abs(np.corrcoef(a[0, :-lag], a[0, lag:])[0, 1]) < lim
    b = noise_block(oracle, 4, 4, range(1), range(0, 8000))
    assert abs(np.corrcoef(a[0], b[0])[0, 1]) < lim
    c = noise_block(oracle, 5, 3, range(1), range(0, 8000))
    assert abs(np.corrcoef(a[0], c[0])[0, 1]) < lim


def test_noise_box_muller_partners_share_a_radius(oracle):
    """Columns 2m and 2m+1 of one worker are the cosine and sine of one pair, so
    their squared sum is -2 ln(u) for a 16-bit bin centre u."""
    for c in range(0, 400, 2):
        r2 = oracle.noise(9, 2, 5, c) ** 2 + oracle.noise(9, 2, 5, c + 1) ** 2
        k = 65536.0 * math.exp(-r2 / 2) - 0.5
        assert abs(k - round(k)) < 1e-6 and 0 <= round(k) < 65536


def test_noise_is_a_pure_function(oracle):
    assert oracle.noise(1, 2, 3, 4) == oracle.noise(1, 2, 3, 4)
    assert oracle.noise(1, 2, 3, 4) != oracle.noise(1, 2 + (1 << 32), 3, 4)


def test_round_count_is_honoured(oracle):
    """Ten rounds are seven rounds followed by three more under the advanced key: ties the reduced-round
    generator of the gradient noise to the known-answer vectors of the ten-round one."""
    weyl = (0x9E3779B9, 0xBB67AE85)
    for ctr, key, want in read_kat():
        assert list(oracle.philox4x32(ctr, key, 10)) == want
        mid = oracle.philox4x32(ctr, key, 7)
        later_key = [(key[0] + 7 * weyl[0]) & 0xFFFFFFFF, (key[1] + 7 * weyl[1]) & 0xFFFFFFFF]
        assert list(oracle.philox4x32(mid, later_key, 3)) == want
        assert list(mid) != want and list(oracle.philox4x32(ctr, key, 6)) != list(mid)
    assert oracle.philox4x32([1, 2, 3, 4], [5, 6], 0) == (1, 2, 3, 4)
