"""Seeded synthetic inputs for the gossip round: the only module that both the
CUDA tests/benchmark and the CPU oracle's tests draw inputs from.

It holds no arithmetic of the method (no mask, no averaging, no peer
selection): only random model/gradient matrices shaped like the flat parameter
vectors of the paper's CNN workloads (Table 2 gives their sizes; Section IV-D
the uniformly random link bandwidths), bandwidth matrices and matchings.
Everything is numpy on the host, keyed by an explicit seed.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One benchmark/parity configuration."""
    name: str
    n: int                       # workers
    N: int                       # parameters per worker
    x_std: float                 # model entries ~ N(0, x_std)
    g_std: float                 # gradient entries ~ N(0, g_std)
    lr: float
    keep_fracs: tuple            # 1/c values to run
    rounds: int
    seed: int                    # library seed (mask) and input seed
    pairing: str                 # "fixed" | "select" | "random"
    bw_range: tuple = (1.0, 100.0)   # Mb/s, for pairing == "select"
    fixed_pairs: tuple = field(default=())


WORKLOADS = {
    "tiny": Workload("tiny", 4, 65_536, 1.0, 0.01, 0.1, (0.1,), 3, 0, "fixed",
                     fixed_pairs=(1, 0, 3, 2)),
    "resnet20": Workload("resnet20", 32, 272_474, 0.05, 0.01, 0.1, (0.01,), 100, 1, "select"),
    # the paper's own model sizes (Table 2) with its c = 100
    "mnistcnn": Workload("mnistcnn", 32, 6_653_628, 0.05, 0.01, 0.05, (0.01,), 50, 0, "select"),
    "cifar10cnn": Workload("cifar10cnn", 32, 7_025_886, 0.05, 0.01, 0.04, (0.01,), 50, 0, "select"),
    "vgg16": Workload("vgg16", 32, 14_728_266, 0.05, 0.01, 0.05, (0.01, 0.001), 50, 0, "select"),
    "resnet50": Workload("resnet50", 32, 25_557_032, 0.05, 0.01, 0.05,
                         (0.1, 0.03, 0.01, 0.003, 0.001), 20, 2, "random"),
    "gpt2s": Workload("gpt2s", 32, 124_439_808, 0.02, 0.01, 0.05, (0.01,), 10, 0, "select",
                      bw_range=(1.0, 1000.0)),
}


def gaussian_matrix(n: int, N: int, std: float, seed: int, stream: int = 0) -> np.ndarray:
    """[n, N] float32, entries N(0, std); row i depends only on (seed, stream, i)."""
    out = np.empty((n, N), dtype=np.float32)
    for i in range(n):
        rng = np.random.Generator(np.random.PCG64([seed, stream, i]))
        rng.standard_normal(N, dtype=np.float32, out=out[i])
    out *= np.float32(std)
    return out


def model_and_grad(w: Workload, seed: int | None = None):
    s = w.seed if seed is None else seed
    return gaussian_matrix(w.n, w.N, w.x_std, s, 0), gaussian_matrix(w.n, w.N, w.g_std, s, 1)


def bandwidth_matrix(n: int, lo: float, hi: float, seed: int) -> np.ndarray:
    """Symmetric [n, n] float64 with upper triangle ~ U[lo, hi], zero diagonal."""
    rng = np.random.Generator(np.random.PCG64([seed, 77]))
    B = np.zeros((n, n), dtype=np.float64)
    for i in range(n):
        for j in range(i + 1, n):
            B[i, j] = B[j, i] = rng.uniform(lo, hi)
    return B


def random_perfect_matching(n: int, rng: np.random.Generator) -> np.ndarray:
    """Uniformly random pairing: shuffle, then pair consecutive entries.  With odd
    n the last worker keeps itself."""
    perm = rng.permutation(n)
    pairs = np.arange(n, dtype=np.int32)
    for a in range(0, n - 1, 2):
        i, j = int(perm[a]), int(perm[a + 1])
        pairs[i], pairs[j] = j, i
    return pairs


def hypercube_pairs(n: int, r: int) -> np.ndarray:
    """Round r of the hypercube schedule: worker i talks to i XOR 2^r (n a power of two)."""
    assert n & (n - 1) == 0 and (1 << r) < n
    return np.array([i ^ (1 << r) for i in range(n)], dtype=np.int32)


def matching_rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([seed, 4242]))
