"""Seeded synthetic inputs for the EF21 hot path.

This module only *makes inputs*: feature matrices, labels, shard boundaries,
supplied gradient vectors and the scalar hyper-parameters (k, gamma, lambda).
It contains none of the method's arithmetic (no loss, no gradient, no Top-k,
no state update) so that both the CUDA library and the CPU oracle can take
their inputs from it without sharing any code of the method itself.

The workloads stand in for the LibSVM data sets the paper's logistic
experiments use (Section 5, Table 2: mushrooms, a9a, w8a split over n = 20
clients), which are not available here: shapes, feature density and label
structure follow the paper's table, the values are drawn from a seeded
generator.

Recipe (numpy ``Generator(PCG64(seed))``, draw order fixed):
  1. planted model  w* ~ N(0, I_d)
  2. features       A  (row-major, N x d, float32)
  3. labels         y = sign(A w*) with sign(0) = +1, then each label is
                    flipped independently with probability ``flip``
  4. optional stable sort of the rows by label (-1 first) for a
     heterogeneous split
  5. shards         floor(N/n) rows each, the remainder goes to the last
                    worker (Section 5.1)
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np


@dataclasses.dataclass
class LogisticWorkload:
    """One logistic-regression EF21 problem: shards, labels and scalars."""
    name: str
    n: int
    d: int
    k: int
    gamma: float          # already rounded to float32
    lam: float            # regulariser weight lambda (Section 5, "lambda = 0.1")
    T: int
    A: np.ndarray         # float32 [N, d], row-major, C-contiguous
    y: np.ndarray         # float32 [N], entries +-1
    row_offsets: np.ndarray  # int64 [n+1]
    x0: np.ndarray        # float32 [d]
    seed: int

    @property
    def N(self) -> int:
        return int(self.A.shape[0])


@dataclasses.dataclass
class StressWorkload:
    """Supplied-gradient EF21 problem (no shards): V[n][d] is used at every step."""
    name: str
    n: int
    d: int
    k: int
    gamma: float
    T: int
    seed: int

    def worker_vector(self, i: int) -> np.ndarray:
        return stress_vector(self.seed, i, self.d)

    def all_vectors(self) -> np.ndarray:
        V = np.empty((self.n, self.d), dtype=np.float32)
        for i in range(self.n):
            V[i] = self.worker_vector(i)
        return V


def shard_offsets(N: int, n: int) -> np.ndarray:
    """floor(N/n) rows per worker, remainder to the last one (Section 5.1)."""
    m = N // n
    off = np.arange(n + 1, dtype=np.int64) * m
    off[n] = N
    return off


def _planted_labels(rng: np.random.Generator, A: np.ndarray, w: np.ndarray, flip: float) -> np.ndarray:
    z = A.astype(np.float64) @ w
    y = np.where(z >= 0.0, 1.0, -1.0)
    flips = rng.random(A.shape[0]) < flip
    y = np.where(flips, -y, y)
    return y.astype(np.float32)


def smoothness_constants(A: np.ndarray, row_offsets: np.ndarray, lam: float, objective: str = "logistic") -> np.ndarray:
    """Upper bounds L_i on the gradient-Lipschitz constants of the local losses.

    For the logistic term the curvature of log(1+exp(-t)) is at most 1/4, so the
    Hessian of the mean loss on shard i is bounded by A_i^T A_i / (4 m_i); the
    second derivative of lam*x^2/(1+x^2) is bounded by 2*lam in magnitude.
    These are the L_i of Assumption 1; they are only used to pick a stepsize.
    """
    n = len(row_offsets) - 1
    L = np.zeros(n, dtype=np.float64)
    for i in range(n):
        Ai = A[row_offsets[i]:row_offsets[i + 1]].astype(np.float64)
        m = Ai.shape[0]
        if m == 0:
            L[i] = 2.0 * lam
            continue
        gram = Ai.T @ Ai
        curvature = 0.25 if objective == "logistic" else 2.0      # second derivative bound of the loss in the margin
        L[i] = curvature * float(np.linalg.eigvalsh(gram)[-1]) / m + 2.0 * lam
    return L


def gamma_one_over_L(A: np.ndarray, row_offsets: np.ndarray, lam: float, objective: str = "logistic") -> float:
    """gamma = 1/L with L = mean_i L_i (the bound L <= (1/n) sum L_i of Section 3.3)."""
    L = smoothness_constants(A, row_offsets, lam, objective)
    return float(np.float32(1.0 / float(np.mean(L))))


def theory_gamma(A: np.ndarray, row_offsets: np.ndarray, lam: float, k: int) -> float:
    """Largest stepsize Theorem 1 allows: 1/(L + Ltilde*sqrt(beta/theta)), alpha = k/d."""
    d = A.shape[1]
    L_i = smoothness_constants(A, row_offsets, lam)
    L = float(np.mean(L_i))
    Lt = float(np.sqrt(np.mean(L_i ** 2)))
    alpha = k / d
    if alpha >= 1.0:
        ratio = 0.0
    else:
        r = math.sqrt(1.0 - alpha)
        ratio = r / (1.0 - r)
    return 1.0 / (L + Lt * ratio)


def make_logistic(name: str, n: int, d: int, N: int, k: int, *, seed: int, features: str,
                  density: float = 0.0, const_col: bool = False, flip: float = 0.05,
                  sort_by_label: bool = False, gamma: Optional[float] = None,
                  lam: float = 0.1, T: int = 100) -> LogisticWorkload:
    rng = np.random.default_rng(np.random.PCG64(seed))
    w = rng.standard_normal(d)
    if features == "gauss":
        A = rng.standard_normal((N, d)).astype(np.float32)
    elif features == "bernoulli":
        A = (rng.random((N, d)) < density).astype(np.float32)
        if const_col:
            A[:, d - 1] = 1.0
    else:
        raise ValueError(features)
    y = _planted_labels(rng, A, w, flip)
    if sort_by_label:
        order = np.argsort(y, kind="stable")
        A = np.ascontiguousarray(A[order])
        y = np.ascontiguousarray(y[order])
    off = shard_offsets(N, n)
    if gamma is None:
        gamma = gamma_one_over_L(A, off, lam)
    gamma = float(np.float32(gamma))
    return LogisticWorkload(name=name, n=n, d=d, k=k, gamma=gamma, lam=lam, T=T,
                            A=np.ascontiguousarray(A), y=y, row_offsets=off,
                            x0=np.zeros(d, dtype=np.float32), seed=seed)


def stress_vector(seed: int, i: int, d: int) -> np.ndarray:
    """Worker i's supplied gradient: Student-t(3) entries times a scale s_i ~ U(0.5, 2).

    Every worker has its own stream so that a single worker's vector can be
    regenerated without drawing the others.
    """
    rng = np.random.default_rng(np.random.PCG64([seed, i]))
    s = rng.uniform(0.5, 2.0)
    v = rng.standard_t(3.0, size=d)
    return (v * s).astype(np.float32)


# ---------------------------------------------------------------------------
# The five named workloads.
# ---------------------------------------------------------------------------

def config(index: int, k: Optional[int] = None, scale: float = 1.0):
    """Workload ``index`` (0..4).  ``k`` overrides the default Top-k size
    (workload 2 is run with k in {1, 4, 16}); ``scale`` < 1 shrinks the
    stress workload for tests."""
    if index == 0:
        return make_logistic("tiny", n=4, d=64, N=200, k=k or 4, seed=0, features="gauss",
                             flip=0.10, gamma=0.1, T=100)
    if index == 1:
        return make_logistic("mushrooms-shaped", n=20, d=112, N=8124, k=k or 1, seed=1,
                             features="bernoulli", density=0.19, const_col=True, flip=0.05, T=2000)
    if index == 2:
        return make_logistic("a9a-shaped", n=20, d=123, N=32561, k=k or 1, seed=2,
                             features="bernoulli", density=0.11, flip=0.10, T=2000)
    if index == 3:
        return make_logistic("w8a-shaped", n=20, d=300, N=49749, k=k or 1, seed=3,
                             features="bernoulli", density=0.04, flip=0.05, sort_by_label=True,
                             T=2000)
    if index == 4:
        d = int(4194304 * scale)
        n = 64 if scale == 1.0 else max(2, int(64 * min(1.0, scale * 8)))
        return StressWorkload("topk-stress", n=n, d=d, k=k or max(1, d // 1000), gamma=0.01,
                              T=50, seed=4)
    raise ValueError(f"no workload {index}")


def hbm_scale_logistic(N: int = 500_000):
    """Rows shaped like workload 3 (d = 300, Bernoulli(0.04) features, planted labels with 5 % flips, n = 20 equal
    shards) but N of them, so that the shards (4*N*300 bytes; 600 MB by default) no longer fit in L2 and every
    iteration streams them from HBM.  Same generator and stepsize rule as the other logistic workloads."""
    return make_logistic("w8a-shaped rows beyond L2", n=20, d=300, N=N, k=1, seed=5, features="bernoulli",
                         density=0.04, flip=0.05, T=50)


def minibatch_rows(seed: int, step: int, row_offsets: np.ndarray, tau: int) -> np.ndarray:
    """Rows of one stochastic step: for every worker tau distinct row numbers inside its shard (sampling
    without replacement, as in the paper's minibatch experiments), int32 [n, tau], from its own stream."""
    rng = np.random.default_rng(np.random.PCG64([seed, 7919, step]))
    n = len(row_offsets) - 1
    out = np.empty((n, tau), dtype=np.int32)
    for i in range(n):
        m = int(row_offsets[i + 1] - row_offsets[i])
        out[i] = rng.choice(m, size=tau, replace=False)
    return out


def randk_sets(seed: int, steps: int, n: int, d: int, k: int) -> np.ndarray:
    """Index sets of the Rand-k compressor: for every step and worker k distinct coordinates drawn uniformly
    (sampling without replacement), in ascending order, int32 [steps, n, k]."""
    rng = np.random.default_rng(np.random.PCG64([seed, 104729]))
    out = np.empty((steps, n, k), dtype=np.int32)
    for t in range(steps):
        for i in range(n):
            out[t, i] = np.sort(rng.choice(d, size=k, replace=False))
    return out
