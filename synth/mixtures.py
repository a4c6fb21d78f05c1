"""Gaussian-mixture workloads shaped like the paper's synthetic benchmarks.

The paper evaluates on balanced Gaussian mixtures (its simulation-benchmark
section and the table of (n, d, K, r) settings) and on two real data sets that
are not redistributable here.  Work per iteration depends only on (n, d, r), so
seeded mixtures of the same shapes stand in for all of them.

Everything is generated block by block from independent counter-style streams
(`default_rng([seed, tag, block])`), so any row range can be regenerated without
the rest and the result does not depend on the number of worker threads.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_BLOCK = 1 << 18  # rows per generation block


@dataclasses.dataclass(frozen=True)
class MixtureSpec:
    name: str
    n: int
    d: int
    K: int
    sizes: str            # "equal" | "dirichlet5"
    centre_var: float     # centres ~ N(0, centre_var * I); <0 => uniform on the unit sphere
    noise: str            # "unit" | "percluster" (variance ~ U[0.5, 2]) | "sphere0.3"
    iters: int
    seed: int = 0

    def with_n(self, n: int, name: str | None = None) -> "MixtureSpec":
        """A reduced-n twin: same d, K and distribution."""
        return dataclasses.replace(self, n=int(n), name=name or f"{self.name}-n{n}")


CONFIGS = (
    MixtureSpec("tiny", 2_000, 16, 4, "equal", 25.0, "unit", 200),
    MixtureSpec("medium", 1_000_000, 128, 16, "dirichlet5", 9.0, "unit", 100),
    MixtureSpec("many-cluster", 10_000_000, 64, 100, "equal", 16.0, "percluster", 50),
    MixtureSpec("embedding", 2_000_000, 768, 1000, "equal", -1.0, "sphere0.3", 30),
    MixtureSpec("massive", 100_000_000, 32, 8, "equal", 16.0, "unit", 30),
)


def config(i: int) -> MixtureSpec:
    """1-based index into the five benchmark shapes."""
    return CONFIGS[i - 1]


def default_hparams(K: int) -> dict:
    """Hyper-parameters used for measurement and parity.

    The paper leaves the step size, penalty and tolerances "configurable"; these
    are this build's fixed choices: beta = 1, alpha = 3 / (2 + beta (6K + 2))
    (three times the sufficient step of the paper's smoothness bound at y = 0),
    eps_d = 0.05 for K <= 4 else 0.01, eps_c = 1e-4, T_min = 10.
    """
    beta = 1.0
    alpha = 3.0 / (2.0 + beta * (6.0 * K + 2.0))
    return dict(alpha=float(np.float32(alpha)), beta=float(np.float32(beta)),
                eps_d=0.05 if K <= 4 else 0.01, eps_c=1e-4, T_min=10)


def _cluster_sizes(spec: MixtureSpec, rng: np.random.Generator) -> np.ndarray:
    n, K = spec.n, spec.K
    if spec.sizes == "equal":
        base = np.full(K, n // K, dtype=np.int64)
        base[: n - base.sum()] += 1
        return base
    if spec.sizes == "dirichlet5":
        w = rng.dirichlet(np.full(K, 5.0))
        raw = w * (n - K)                     # every cluster keeps at least one point
        sizes = np.floor(raw).astype(np.int64)
        rem = (n - K) - sizes.sum()
        order = np.argsort(-(raw - sizes), kind="stable")
        sizes[order[:rem]] += 1               # largest-remainder rounding
        return sizes + 1
    raise ValueError(spec.sizes)


def _centres(spec: MixtureSpec, rng: np.random.Generator) -> np.ndarray:
    g = rng.standard_normal((spec.K, spec.d))
    if spec.centre_var < 0:
        return (g / np.linalg.norm(g, axis=1, keepdims=True)).astype(np.float32)
    return (np.sqrt(spec.centre_var) * g).astype(np.float32)


def _workers() -> int:
    return max(1, min(16, os.cpu_count() or 1))


def make_mixture(spec: MixtureSpec, out: np.ndarray | None = None, rows: int | None = None):
    """Return (X, labels, centres): X is n x d float32 row-major, labels int32.

    Labels are contiguous blocks of the cluster sizes followed by a seeded row
    shuffle, so cluster membership is spread over the whole row range.
    With `rows` only the leading rows of the same problem are generated (X and
    labels are cut to `rows`; the values equal those of the full problem).
    """
    n, d, K = spec.n, spec.d, spec.K
    head = np.random.default_rng([spec.seed, 0])
    sizes = _cluster_sizes(spec, head)
    centres = _centres(spec, head)
    if spec.noise == "percluster":
        sigma = np.sqrt(head.uniform(0.5, 2.0, size=K)).astype(np.float32)
    elif spec.noise == "sphere0.3":
        sigma = np.full(K, 0.3, dtype=np.float32)
    else:
        sigma = np.ones(K, dtype=np.float32)
    labels = np.repeat(np.arange(K, dtype=np.int32), sizes)
    np.random.default_rng([spec.seed, 1]).shuffle(labels)
    if rows is not None:
        n = min(n, int(rows))
        labels = labels[:n]
    X = out if out is not None else np.empty((n, d), dtype=np.float32)
    assert X.shape == (n, d) and X.dtype == np.float32 and X.flags.c_contiguous

    def fill(b: int) -> None:
        lo, hi = b * _BLOCK, min(n, (b + 1) * _BLOCK)
        rng = np.random.default_rng([spec.seed, 2, b])
        z = rng.standard_normal((hi - lo, d), dtype=np.float32)
        lab = labels[lo:hi]
        z *= sigma[lab][:, None]
        z += centres[lab]
        if spec.noise == "sphere0.3":
            z /= np.linalg.norm(z, axis=1, keepdims=True)
        X[lo:hi] = z

    nblocks = (n + _BLOCK - 1) // _BLOCK
    if nblocks == 1:
        fill(0)
    else:
        with ThreadPoolExecutor(_workers()) as ex:
            list(ex.map(fill, range(nblocks)))
    return X, labels, centres


def make_u0(n: int, r: int, K: int, seed: int = 0, out: np.ndarray | None = None) -> np.ndarray:
    """Starting factor: i.i.d. U(0,1) entries rescaled so that ||U0||_F^2 = K.

    Nonnegativity and the Frobenius radius are the two constraints of the
    feasible set that a rescaling can impose; the row-sum constraint is what
    the iteration itself drives to zero.
    """
    U = out if out is not None else np.empty((n, r), dtype=np.float32)
    nblocks = (n + _BLOCK - 1) // _BLOCK
    ss = np.zeros(nblocks, dtype=np.float64)

    def fill(b: int) -> None:
        lo, hi = b * _BLOCK, min(n, (b + 1) * _BLOCK)
        rng = np.random.default_rng([seed, 3, b])
        z = rng.random((hi - lo, r), dtype=np.float32)
        U[lo:hi] = z
        ss[b] = float(np.sum(z.astype(np.float64) ** 2))

    def scale(b: int, c: np.float32) -> None:
        lo, hi = b * _BLOCK, min(n, (b + 1) * _BLOCK)
        U[lo:hi] *= c

    if nblocks == 1:
        fill(0)
        scale(0, np.float32(np.sqrt(K / ss.sum())))
    else:
        with ThreadPoolExecutor(_workers()) as ex:
            list(ex.map(fill, range(nblocks)))
            c = np.float32(np.sqrt(K / ss.sum()))
            list(ex.map(lambda b: scale(b, c), range(nblocks)))
    return U


def separated_tiny_mixture(n: int, K: int, d: int = 3, sep: float = 10.0, sigma: float = 0.5,
                           seed: int = 0):
    """n <= 12 points in K well-separated groups, for brute-force exact K-means.

    Centres sit on coordinate axes `sep` apart from the origin (pairwise distance
    sqrt(2) * sep), group sizes as equal as possible, rows shuffled.
    """
    assert K <= d
    rng = np.random.default_rng([seed, 4])
    centres = np.zeros((K, d))
    for k in range(K):
        centres[k, k] = sep
    sizes = np.full(K, n // K)
    sizes[: n - sizes.sum()] += 1
    labels = np.repeat(np.arange(K, dtype=np.int32), sizes)
    rng.shuffle(labels)
    X = centres[labels] + sigma * rng.standard_normal((n, d))
    return X.astype(np.float32), labels
