"""Pins for the oracle's run loops: Algorithm 1's `for t = 1, ..., T`.

`oracle.run(t0, steps)` has to be `steps` single iterations with the step index
t0, t0 + 1, ..., t0 + steps - 1 (the index is 0-based and enters the drop masks
and the gradient noise through the Philox counter), each starting from the state
the one before left.  Every free-running comparison of the CUDA path takes its
expected values from these loops, so they are tied here, on the CPU, to the
single step, which has pins of its own (X_{t+1} = V_t W_t of Eq. 3 and the closed
forms).  A loop that starts one step late, repeats a step index or skips one
fails: with noise and drops on, two different step indices give different bits.
None of these tests touches the CUDA library.
"""
import numpy as np
import pytest

from paper_1810_07766_b200 import workloads as wl


def _state(n, d, dtype, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, d)).astype(np.float32)
    b = rng.standard_normal((n, d)).astype(np.float32)
    if dtype == "bf16":
        return wl.f32_to_bf16_bits(x), wl.f32_to_bf16_bits(b)
    return x, b


@pytest.mark.parametrize("average_gradients", [False, True])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("t0", [0, 5, 2**32 - 2])
def test_run_is_repeated_single_steps_with_consecutive_step_indices(oracle, average_gradients, dtype, t0):
    n, d, steps = 5, 37, 4
    kw = dict(dtype=dtype, gamma=0.07, sigma=0.2, p=0.3, seed=0xC0FFEE123, assign=oracle.ASSIGN_PERM,
              average_gradients=average_gradients)
    x0, b = _state(n, d, dtype, 11)
    ran = x0.copy()
    oracle.run(ran, b, t0=t0, steps=steps, **kw)
    stepped = x0.copy()
    for k in range(steps):
        oracle.step(stepped, b, t=t0 + k, **kw)
    assert np.array_equal(ran.view(np.uint8), stepped.view(np.uint8))

    # the comparison can tell the step indices apart: a run that starts one step late, or that uses
    # t0 for every step, ends somewhere else
    late = x0.copy()
    for k in range(steps):
        oracle.step(late, b, t=t0 + k + 1, **kw)
    stuck = x0.copy()
    for k in range(steps):
        oracle.step(stuck, b, t=t0, **kw)
    assert not np.array_equal(ran.view(np.uint8), late.view(np.uint8))
    assert not np.array_equal(ran.view(np.uint8), stuck.view(np.uint8))


@pytest.mark.parametrize("average_gradients", [False, True])
def test_a_run_can_be_cut_anywhere(oracle, average_gradients):
    # T steps at once = k steps, then T - k from step index t0 + k: the loop carries nothing but x and t
    n, d, t0, steps = 4, 23, 2**32 - 3, 7
    kw = dict(dtype="f32", gamma=0.05, sigma=0.1, p=0.2, seed=99, average_gradients=average_gradients)
    x0, b = _state(n, d, "f32", 5)
    whole = x0.copy()
    oracle.run(whole, b, t0=t0, steps=steps, **kw)
    for cut in (0, 1, 3, steps):
        parts = x0.copy()
        oracle.run(parts, b, t0=t0, steps=cut, **kw)
        oracle.run(parts, b, t0=t0 + cut, steps=steps - cut, **kw)
        assert np.array_equal(whole, parts), cut


def test_zero_steps_change_nothing(oracle):
    x0, b = _state(3, 9, "f32", 1)
    for avg in (False, True):
        x = x0.copy()
        oracle.run(x, b, dtype="f32", gamma=0.1, sigma=0.1, p=0.5, seed=1, t0=17, steps=0, average_gradients=avg)
        assert np.array_equal(x, x0)


@pytest.mark.parametrize("average_gradients", [False, True])
def test_run_without_noise_and_drops_follows_the_closed_form(oracle, average_gradients):
    # p = 0, sigma = 0, common start 0: every replica is (1 - (1 - gamma)^T) mean_i b_i after T steps,
    # whichever of the two quantities is averaged; a loop that ran T - 1 or T + 1 steps misses it.
    n, d, gamma, steps = 4, 16, 0.125, 6
    rng = np.random.default_rng(3)
    b = rng.standard_normal((n, d)).astype(np.float32)
    x = np.zeros((n, d), dtype=np.float32)
    oracle.run(x, b, dtype="f32", gamma=gamma, sigma=0.0, p=0.0, seed=7, t0=40, steps=steps,
               average_gradients=average_gradients)
    want = (1.0 - (1.0 - gamma) ** steps) * b.astype(np.float64).mean(axis=0)
    assert np.max(np.abs(x - want[None, :])) < 2e-6
    off_by_one = (1.0 - (1.0 - gamma) ** (steps + 1)) * b.astype(np.float64).mean(axis=0)
    assert np.max(np.abs(x - off_by_one[None, :])) > 1e-3
