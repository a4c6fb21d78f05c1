"""One NLR iteration (Algorithm 1) restated with numpy in FP64, row-chunked, with BLAS matrix
products as the library primitive.  Test infrastructure: it exists so that the largest benchmark
shape (n = 2e6, d = 768, K = 1000: about 6 TFLOP per iteration), which the plain C oracle needs
minutes for, can still be checked on every entry.  It follows the same steps and the same rounding
points as the C oracle (FP32 buffers, FP64 sums, one rounding per stored value) and is pinned
against it on small problems by the CPU tests.
"""
from __future__ import annotations

import numpy as np


def iteration(Xhat: np.ndarray, U: np.ndarray, ytilde: np.ndarray, K: int, alpha: float, beta: float,
              eps_d: float, dual_pending: bool = False, rows: int = 1 << 16):
    """(U_new FP32, ytilde_new FP32, info) from the iterate (U, ytilde) the iteration starts from.

    Steps (Algorithm 1, with the call-by-call detail of Algorithm 2):
      p = U^T 1, q = U p - 1, [gated ytilde += gamma q of the previous iteration], ybar = ytilde + gamma q,
      s = U^T ybar, Theta = Xhat^T U, W = [U + 2 alpha Xhat Theta - alpha (ybar p^T + 1 s^T)]_+,
      a = sum W^2, b = sum U^2, h = sum W U, c = FP32(sqrt(K) / sqrt(a)), U_new = FP32(c W),
      Delta = max(c^2 a + b - 2 c h, 0), delta_hat = sqrt(Delta) / sqrt(K), gate = Delta < eps_d^2 K.
    """
    n, d = Xhat.shape
    r = U.shape[1]
    gamma = float(beta) / n
    alpha32 = np.float32(alpha)
    # p, q
    p64 = np.zeros(r)
    for lo in range(0, n, rows):
        p64 += U[lo:lo + rows].astype(np.float64).sum(axis=0)
    p = p64.astype(np.float32)
    q = np.empty(n, np.float32)
    for lo in range(0, n, rows):
        q[lo:lo + rows] = (U[lo:lo + rows].astype(np.float64) @ p.astype(np.float64) - 1.0).astype(np.float32)
    yt = np.array(ytilde, dtype=np.float32, copy=True)
    if dual_pending:
        yt = (yt.astype(np.float64) + gamma * q.astype(np.float64)).astype(np.float32)
    ybar = (yt.astype(np.float64) + gamma * q.astype(np.float64)).astype(np.float32)
    # s, Theta
    s64 = np.zeros(r)
    th64 = np.zeros((d, r))
    for lo in range(0, n, rows):
        Uc = U[lo:lo + rows].astype(np.float64)
        s64 += Uc.T @ ybar[lo:lo + rows].astype(np.float64)
        th64 += Xhat[lo:lo + rows].astype(np.float64).T @ Uc
    s = s64.astype(np.float32)
    Theta = th64.astype(np.float32)
    fhat = -float((th64 ** 2).sum()) + float(yt.astype(np.float64) @ q.astype(np.float64)) \
        + 0.5 * gamma * float(q.astype(np.float64) @ q.astype(np.float64))
    # W and the statistics
    W = np.empty((n, r), np.float32)
    a = b = h = 0.0
    th_d, p_d, s_d = Theta.astype(np.float64), p.astype(np.float64), s.astype(np.float64)
    al = float(alpha32)
    for lo in range(0, n, rows):
        Uc = U[lo:lo + rows].astype(np.float64)
        G = Xhat[lo:lo + rows].astype(np.float64) @ th_d
        V = Uc + 2.0 * al * G - al * (np.outer(ybar[lo:lo + rows].astype(np.float64), p_d) + s_d[None, :])
        Wc = np.maximum(V, 0.0).astype(np.float32)
        W[lo:lo + rows] = Wc
        Wd = Wc.astype(np.float64)
        a += float((Wd * Wd).sum())
        b += float((Uc * Uc).sum())
        h += float((Wd * Uc).sum())
    nu = np.sqrt(a)
    info = dict(a=a, b=b, h=h, fhat=fhat, status=0)
    if not nu > 1e-20:
        info["status"] = -4
        return W, yt, info
    c_f = np.float32(np.sqrt(float(K)) / nu)
    c = float(c_f)
    for lo in range(0, n, rows):
        W[lo:lo + rows] *= c_f
    Delta = max(c * c * a + b - 2.0 * c * h, 0.0)
    info.update(c=c, Delta=Delta, delta_hat=float(np.sqrt(Delta) / np.sqrt(float(K))),
                dual=int(Delta < eps_d * eps_d * K))
    return W, yt, info
