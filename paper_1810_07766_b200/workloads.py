"""Seeded synthetic inputs for the RPS synchronisation step.

This module only *generates inputs* (the per-worker targets ``b_i`` of the
quadratic objective ``f_i(x) = 0.5 * ||x - b_i||^2`` and the scalar settings of
each workload).  It contains none of the method's arithmetic: no SGD update, no
drop masks, no averaging, no Philox.  Both the CUDA path and the CPU oracle are
handed the arrays produced here, so neither side ever consumes a value computed
by the other.

The workloads stand in for the flat parameter vectors of the networks the paper
trains (Section 5: ResNets on CIFAR-10, an LSTM on ATIS); only the vector's size
matters to the synchronisation step, so the sizes are ResNet-18- and
ResNet-50-like flat vectors, a prime-ish size with a ragged last block, and a
bf16 case.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One configuration of Algorithm 1's inputs plus the synthetic objective."""

    name: str
    n: int                 # workers == parameter servers == blocks
    d: int                 # flat model size
    dtype: str             # "f32" or "bf16" (replica storage type)
    p: float               # packet drop probability (Section 3)
    gamma: float           # learning rate
    sigma: float           # std-dev of the Gaussian gradient noise
    seed: int
    steps: int             # T
    hetero: bool = False   # b_i ~ N(mu_i, 1) with mu_i ~ U(-1, 1) instead of N(0, 1)
    p_sweep: Tuple[float, ...] = ()

    @property
    def replica_params(self) -> int:
        return self.n * self.d

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def bytes_per_step(self) -> int:
        """Algorithmic HBM traffic of one step: read x, read b, write x."""
        return 3 * self.elem_bytes * self.n * self.d

    def scaled(self, d: int, steps: int | None = None) -> "Workload":
        """Same workload on a shorter vector (used by parity tests)."""
        return replace(self, d=d, steps=self.steps if steps is None else steps,
                       name=f"{self.name}@d={d}")


WORKLOADS = {
    "cfg1": Workload("cfg1", n=4, d=65_536, dtype="f32", p=0.1, gamma=0.1, sigma=0.1,
                     seed=0, steps=100),
    "cfg2": Workload("cfg2", n=8, d=11_173_962, dtype="f32", p=0.1, gamma=0.05, sigma=0.1,
                     seed=1, steps=50, p_sweep=(0.0, 0.01, 0.05, 0.1, 0.2)),
    "cfg3": Workload("cfg3", n=16, d=25_557_032, dtype="f32", p=0.1, gamma=0.05, sigma=0.1,
                     seed=2, steps=200, hetero=True),
    "cfg4": Workload("cfg4", n=32, d=4_000_037, dtype="f32", p=0.1, gamma=0.1, sigma=0.05,
                     seed=3, steps=50, p_sweep=(0.05, 0.1, 0.2, 0.3)),
    "cfg5": Workload("cfg5", n=64, d=16_777_216, dtype="bf16", p=0.05, gamma=0.02, sigma=0.1,
                     seed=4, steps=100),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (round-to-nearest-even), returned as uint16 bits."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_targets(w: Workload) -> np.ndarray:
    """Targets ``b`` as a dense ``[n][d]`` array.

    float32 for "f32" workloads; uint16 bfloat16 bit patterns for "bf16"
    workloads.  Rows are drawn worker by worker from ``default_rng(seed)`` so a
    prefix of the workers is reproducible on its own.
    """
    rng = np.random.default_rng(w.seed)
    mu = rng.uniform(-1.0, 1.0, size=w.n) if w.hetero else np.zeros(w.n)
    b = np.empty((w.n, w.d), dtype=np.float32)
    for i in range(w.n):
        b[i] = rng.standard_normal(w.d, dtype=np.float32)
        if w.hetero:
            b[i] += np.float32(mu[i])
    if w.dtype == "bf16":
        return f32_to_bf16_bits(b)
    return b


def make_initial(w: Workload) -> np.ndarray:
    """Common initial model of all workers: zero (Assumption 1, item 3)."""
    if w.dtype == "bf16":
        return np.zeros((w.n, w.d), dtype=np.uint16)
    return np.zeros((w.n, w.d), dtype=np.float32)


def as_float64(w: Workload, a: np.ndarray) -> np.ndarray:
    """Numeric view of a replica-typed array as float64 (for comparisons)."""
    if w.dtype == "bf16":
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)
