"""ctypes front end of the CPU oracle (test infrastructure; see nlr_oracle.c).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It never touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nlr_oracle.c")
_LIB = os.path.join(_HERE, "libnlr_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class Info(C.Structure):
    _fields_ = [("t", C.c_int32), ("dual", C.c_int32), ("stop", C.c_int32), ("status", C.c_int32),
                ("a", C.c_double), ("b", C.c_double), ("h", C.c_double), ("c", C.c_double),
                ("Delta", C.c_double), ("delta_hat", C.c_double), ("rho", C.c_double),
                ("fhat", C.c_double)]

    def as_dict(self) -> dict:
        return {k: getattr(self, k) for k, _ in self._fields_}


_F = np.ctypeslib.ndpointer(dtype=np.float32, flags="C_CONTIGUOUS")
_D = np.ctypeslib.ndpointer(dtype=np.float64, flags="C_CONTIGUOUS")
_I = np.ctypeslib.ndpointer(dtype=np.int32, flags="C_CONTIGUOUS")


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.nlr_oracle_threads.restype = C.c_int
        L.nlr_oracle_col_mean.argtypes = [_F, C.c_int64, C.c_int32, _D]
        L.nlr_oracle_gram.argtypes = [_F, C.c_int64, C.c_int32, C.c_void_p, _D]
        L.nlr_oracle_sym_eig_max.argtypes = [_D, C.c_int32]
        L.nlr_oracle_sym_eig_max.restype = C.c_double
        L.nlr_oracle_spectral_norm.argtypes = [_F, C.c_int64, C.c_int32, C.c_int32, _D]
        L.nlr_oracle_spectral_norm.restype = C.c_double
        L.nlr_oracle_normalize.argtypes = [_F, C.c_int64, C.c_int32, _D, C.c_double, _F]
        L.nlr_oracle_residual.argtypes = [_F, C.c_int64, C.c_int32, _F, _F]
        L.nlr_oracle_theta.argtypes = [_F, _F, C.c_int64, C.c_int32, C.c_int32, _F]
        L.nlr_oracle_objective.argtypes = [_F, _F, _F, C.c_int64, C.c_int32, C.c_int32, C.c_double]
        L.nlr_oracle_objective.restype = C.c_double
        L.nlr_oracle_step.argtypes = [_F, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_double,
                                      C.c_double, C.c_double, C.c_double, C.c_int32, C.c_int32,
                                      _F, _F, _F, _F, _F, _F, _F, C.POINTER(Info)]
        L.nlr_oracle_step.restype = C.c_int
        L.nlr_oracle_run.argtypes = [_F, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_double,
                                     C.c_double, C.c_double, C.c_double, C.c_int32, C.c_int32,
                                     _F, _F, C.POINTER(Info), C.POINTER(C.c_int32)]
        L.nlr_oracle_run.restype = C.c_int
        L.nlr_oracle_labels.argtypes = [_F, C.c_int64, C.c_int32, _I]
        L.nlr_oracle_kmeans_cost.argtypes = [_F, C.c_int64, C.c_int32, _I, C.c_int32]
        L.nlr_oracle_kmeans_cost.restype = C.c_double
        _lib = L
    return _lib


def threads() -> int:
    return int(lib().nlr_oracle_threads())


def col_mean(X: np.ndarray) -> np.ndarray:
    n, d = X.shape
    m = np.zeros(d)
    lib().nlr_oracle_col_mean(X, n, d, m)
    return m


def gram(X: np.ndarray, mean: np.ndarray | None) -> np.ndarray:
    n, d = X.shape
    G = np.zeros((d, d))
    ptr = None if mean is None else mean.ctypes.data_as(C.c_void_p)
    lib().nlr_oracle_gram(X, n, d, ptr, G)
    return G


def sym_eig_max(G: np.ndarray) -> float:
    G = np.ascontiguousarray(G, dtype=np.float64)
    return float(lib().nlr_oracle_sym_eig_max(G, G.shape[0]))


def spectral_norm(X: np.ndarray, center: bool = True):
    """Returns (a, mean): a = ||X - 1 mean^T||_2 (mean = 0 when center is False)."""
    n, d = X.shape
    mean = np.zeros(d)
    a = lib().nlr_oracle_spectral_norm(X, n, d, int(center), mean)
    return float(a), mean


def normalize(X: np.ndarray, center: bool = True):
    """Returns (Xhat, a, mean) with Xhat = fp32((X - mean) / a)."""
    a, mean = spectral_norm(X, center)
    Xhat = np.empty_like(X)
    lib().nlr_oracle_normalize(X, X.shape[0], X.shape[1], mean, a, Xhat)
    return Xhat, a, mean


def residual(U: np.ndarray):
    n, r = U.shape
    p = np.empty(r, np.float32)
    q = np.empty(n, np.float32)
    lib().nlr_oracle_residual(U, n, r, p, q)
    return p, q


def theta(Xhat: np.ndarray, U: np.ndarray) -> np.ndarray:
    n, d = Xhat.shape
    r = U.shape[1]
    T = np.empty((d, r), np.float32)
    lib().nlr_oracle_theta(Xhat, U, n, d, r, T)
    return T


def objective(Xhat: np.ndarray, U: np.ndarray, ytilde: np.ndarray, beta: float) -> float:
    n, d = Xhat.shape
    return float(lib().nlr_oracle_objective(Xhat, U, ytilde, n, d, U.shape[1], float(beta)))


class State:
    """Iteration state of Algorithm 1: U, ytilde = y/sqrt(n), p, q and the iteration index."""

    def __init__(self, Xhat: np.ndarray, U0: np.ndarray, ytilde: np.ndarray | None = None, t: int = 0):
        self.Xhat = np.ascontiguousarray(Xhat, np.float32)
        self.U = np.array(U0, dtype=np.float32, order="C", copy=True)
        n, r = self.U.shape
        self.ytilde = (np.zeros(n, np.float32) if ytilde is None
                       else np.array(ytilde, dtype=np.float32, copy=True))
        self.p, self.q = residual(self.U)
        self.Theta = np.zeros((self.Xhat.shape[1], r), np.float32)
        self.ybar = np.zeros(n, np.float32)
        self.s = np.zeros(r, np.float32)
        self.t = t

    def step(self, K: int, alpha: float, beta: float, eps_d: float, eps_c: float, T_min: int) -> dict:
        n, d = self.Xhat.shape
        r = self.U.shape[1]
        info = Info()
        lib().nlr_oracle_step(self.Xhat, n, d, r, K, float(alpha), float(beta), float(eps_d),
                              float(eps_c), int(T_min), int(self.t), self.U, self.ytilde, self.p,
                              self.q, self.Theta, self.ybar, self.s, C.byref(info))
        if info.status == 0:
            self.t += 1
        return info.as_dict()


def run(Xhat: np.ndarray, U0: np.ndarray, K: int, alpha: float, beta: float, eps_d: float,
        eps_c: float, T: int, T_min: int, ytilde: np.ndarray | None = None):
    """Algorithm 1 from (U0, y = 0 unless given). Returns (U, ytilde, last_info, iters, rc)."""
    Xhat = np.ascontiguousarray(Xhat, np.float32)
    U = np.array(U0, dtype=np.float32, order="C", copy=True)
    n, d = Xhat.shape
    r = U.shape[1]
    yt = np.zeros(n, np.float32) if ytilde is None else np.array(ytilde, dtype=np.float32, copy=True)
    info = Info()
    iters = C.c_int32(0)
    rc = lib().nlr_oracle_run(Xhat, n, d, r, K, float(alpha), float(beta), float(eps_d), float(eps_c),
                              int(T), int(T_min), U, yt, C.byref(info), C.byref(iters))
    return U, yt, info.as_dict(), int(iters.value), int(rc)


def labels(U: np.ndarray) -> np.ndarray:
    n, r = U.shape
    out = np.empty(n, np.int32)
    lib().nlr_oracle_labels(np.ascontiguousarray(U, np.float32), n, r, out)
    return out


def kmeans_cost(X: np.ndarray, lab: np.ndarray, K: int) -> float:
    n, d = X.shape
    return float(lib().nlr_oracle_kmeans_cost(np.ascontiguousarray(X, np.float32), n, d,
                                              np.ascontiguousarray(lab, np.int32), K))
