"""Data-informed starting factor (the paper's appendix "Additional Computation Details", paragraph
"Initialization"), restated with numpy in FP64.  TEST INFRASTRUCTURE: only tests may import this; it
shares no code with the CUDA path.

    V = X-hat X-hat^T Z,   V = Q R,   U0 = Proj_Omega(Q)

with the orthonormalization done by Cholesky QR in feature space, in the paper's notation:

    M = X-hat^T Z (d x r),  C = X-hat^T X-hat (d x d),  V^T V = M^T C M = R^T R (R upper triangular),
    Q = X-hat (M R^{-1}),   U0 = sqrt(K) [Q]_+ / ||[Q]_+||_F      (projection onto {U >= 0, ||U||_F^2 = K}).

Z is an input (the method's random draw is the caller's).  Library primitives: matrix products, the Cholesky
factorization and the triangular solve.  Everything is FP64; U0 is rounded once to FP32, the factor's storage
type.  The sample must have full column rank (r <= d and V well conditioned): otherwise the Cholesky
factorization fails, as the paper notes, and `numpy.linalg.LinAlgError` propagates.

Parity pins (tests/test_oracle_pins.py): Q^T Q = I; Q equals the Q factor of a Householder QR of the explicit
X-hat X-hat^T Z up to the sign convention; U0 >= 0 and ||U0||_F^2 = K; the objective at U0 is below the
objective at the uniform random start on planted-mixture data.
"""
from __future__ import annotations

import numpy as np


def range_init(Xhat: np.ndarray, Z: np.ndarray, K: int, rows: int = 1 << 16):
    """Returns (U0 FP32 n x r, info) with info = {"Q": FP64 Q (only when n * r <= 2e7), "R": R, "B": M R^{-1},
    "norm_pos": ||[Q]_+||_F}."""
    n, d = Xhat.shape
    r = Z.shape[1]
    M = np.zeros((d, r))
    C = np.zeros((d, d))
    for lo in range(0, n, rows):                       # row chunks only bound the FP64 temporaries
        Xc = Xhat[lo:lo + rows].astype(np.float64)
        M += Xc.T @ Z[lo:lo + rows].astype(np.float64)
        C += Xc.T @ Xc
    G = M.T @ (C @ M)
    G = 0.5 * (G + G.T)
    R = np.linalg.cholesky(G).T                        # upper triangular, positive diagonal: G = R^T R
    B = np.linalg.solve(R.T, M.T).T                    # B R = M  (triangular system, solved row by row)
    U0 = np.empty((n, r), np.float32)
    ss = 0.0
    keepQ = n * r <= 20_000_000
    Q = np.empty((n, r)) if keepQ else None
    for lo in range(0, n, rows):
        q = Xhat[lo:lo + rows].astype(np.float64) @ B
        if keepQ:
            Q[lo:lo + rows] = q
        w = np.maximum(q, 0.0)
        ss += float(np.sum(w * w))
    nu = np.sqrt(ss)
    c = np.sqrt(float(K)) / nu
    for lo in range(0, n, rows):
        q = Xhat[lo:lo + rows].astype(np.float64) @ B
        U0[lo:lo + rows] = (c * np.maximum(q, 0.0)).astype(np.float32)
    return U0, {"Q": Q, "R": R, "B": B, "norm_pos": nu}
