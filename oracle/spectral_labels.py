"""Label read-out for a factor with more columns than clusters (the paper's appendix "Additional Computation
Details", paragraph "Recover cluster labels from U matrix"), restated with numpy in FP64.  TEST
INFRASTRUCTURE: only tests may import this; it shares no code with the CUDA path.

    U = P S Q^T (singular value decomposition);  Y = the leading K left singular vectors (n x K);
    cluster the rows of Y with K-means.

The paper does not say how its K-means is seeded or stopped.  The reading taken here is deterministic, so that
two implementations can be compared label by label:

  seeding   farthest-point: the first centre is the row of Y with the largest norm, every further centre the
            row with the largest distance to its nearest chosen centre (lowest row index on ties);
  Lloyd     assign every row to the nearest centre (lowest centre index on ties), move every centre to the
            mean of its rows (a centre without rows stays where it is), until no label changes or max_iter
            assignment passes have been made.

Label k is the k-th seeded centre.  Singular vectors are fixed only up to sign, and up to a rotation inside an
eigenspace of equal singular values; distances between rows of Y do not depend on either as long as
sigma_K > sigma_{K+1}, so the partition is well defined.

Parity pins (tests/test_oracle_pins.py): on a factor with exactly constant rows per planted cluster spread over
several columns each (r > K) the planted partition comes back; the Gram route (eigenvectors of U^T U) gives the
same embedding distances as the SVD; the Lloyd result is a fixed point (every row is nearest to its own
centre, every centre is the mean of its rows) and never costs more than the seeding.
"""
from __future__ import annotations

import numpy as np


def embedding(U: np.ndarray, K: int) -> np.ndarray:
    """Leading K left singular vectors of U (n x K, FP64), by the library SVD."""
    P, S, _ = np.linalg.svd(U.astype(np.float64), full_matrices=False)
    return P[:, :K]


def farthest_point_seeds(Y: np.ndarray, K: int) -> np.ndarray:
    """Row indices of the K seeds."""
    n = Y.shape[0]
    norms = np.einsum("ij,ij->i", Y, Y)
    seeds = [int(np.argmax(norms))]                       # argmax returns the lowest index among maxima
    mind = np.full(n, np.inf)
    for _ in range(1, K):
        diff = Y - Y[seeds[-1]]
        mind = np.minimum(mind, np.einsum("ij,ij->i", diff, diff))
        seeds.append(int(np.argmax(mind)))
    return np.array(seeds, dtype=np.int64)


def lloyd(Y: np.ndarray, centres: np.ndarray, max_iter: int = 50):
    """Returns (labels int32, centres, assignment passes made)."""
    n, K = Y.shape[0], centres.shape[0]
    centres = centres.copy()
    labels = np.full(n, -1, dtype=np.int32)
    passes = 0
    for _ in range(max_iter):
        d2 = ((Y[:, None, :] - centres[None, :, :]) ** 2).sum(axis=2) if n * K * Y.shape[1] <= 5e7 else \
            np.stack([np.einsum("ij,ij->i", Y - c, Y - c) for c in centres], axis=1)
        new = np.argmin(d2, axis=1).astype(np.int32)      # lowest centre index on ties
        passes += 1
        changed = int(np.sum(new != labels))
        labels = new
        if changed == 0:
            break
        for k in range(K):
            members = Y[labels == k]
            if members.shape[0]:
                centres[k] = members.mean(axis=0)
    return labels, centres, passes


def spectral_labels(U: np.ndarray, K: int, max_iter: int = 50):
    """Labels (int32, n), the embedding and the number of assignment passes."""
    Y = embedding(U, K)
    seeds = farthest_point_seeds(Y, K)
    labels, centres, passes = lloyd(Y, Y[seeds].copy(), max_iter)
    return labels, Y, passes
