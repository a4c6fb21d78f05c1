"""ctypes binding with the same names as the C ABI (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgemnlr.so")

OK, CONVERGED, ITER_CAP = 0, 1, 2
E_INVALID, E_CUDA, E_WORKSPACE, E_BREAKDOWN, E_NONFINITE, E_NOT_READY = -1, -2, -3, -4, -5, -6
E_TIMEOUT, E_TOO_LARGE = -7, -8
STATIC_MAX_R = 128


class Params(C.Structure):
    """Mirror of gem_nlr_params."""
    _fields_ = [("n", C.c_int64), ("d", C.c_int32), ("K", C.c_int32), ("r", C.c_int32),
                ("alpha", C.c_float), ("beta", C.c_float), ("T", C.c_int32), ("T_min", C.c_int32),
                ("eps_d", C.c_double), ("eps_c", C.c_double), ("center", C.c_int32),
                ("x_inplace", C.c_int32), ("pi_max_iters", C.c_int32), ("pi_tol", C.c_double),
                ("pi_seed", C.c_uint64), ("precision", C.c_int32), ("history", C.c_int32)]


class IterInfo(C.Structure):
    """Mirror of gem_nlr_iter_info."""
    _fields_ = [("t", C.c_int32), ("dual_applied", C.c_int32), ("stop", C.c_int32),
                ("status", C.c_int32), ("a", C.c_double), ("b", C.c_double), ("h", C.c_double),
                ("c", C.c_double), ("delta_hat", C.c_double), ("rho", C.c_double),
                ("fhat", C.c_double)]

    def as_dict(self) -> dict:
        return {k: getattr(self, k) for k, _ in self._fields_}


_lib = None


def library_path() -> str:
    return _LIB_PATH


def lib():
    """Load libgemnlr.so; raises if it has not been built (python -m paper_2609_36074_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                               "`python paper_2609_36074_b200/build.py` (nvcc, sm_100a)")
        L = C.CDLL(_LIB_PATH)
        vp, pp = C.c_void_p, C.POINTER(Params)
        L.gem_nlr_workspace_bytes.argtypes = [pp]
        L.gem_nlr_workspace_bytes.restype = C.c_size_t
        L.gem_nlr_paper_storage_bytes.argtypes = [pp]
        L.gem_nlr_paper_storage_bytes.restype = C.c_size_t
        L.gem_nlr_create.argtypes = [C.POINTER(vp), pp, vp, vp, vp, C.c_size_t, vp]
        L.gem_nlr_spectral_norm.argtypes = [vp, C.POINTER(C.c_double)]
        L.gem_nlr_set_normalized.argtypes = [vp, C.c_double]
        L.gem_nlr_step.argtypes = [vp, C.POINTER(IterInfo)]
        L.gem_nlr_run.argtypes = [vp, C.POINTER(IterInfo), C.POINTER(C.c_int32)]
        L.gem_nlr_labels.argtypes = [vp, vp]
        L.gem_nlr_objective.argtypes = [vp, C.POINTER(C.c_double)]
        L.gem_nlr_get_state.argtypes = [vp, vp, C.POINTER(C.c_int32)]
        L.gem_nlr_set_state.argtypes = [vp, vp, C.c_int32]
        L.gem_nlr_history.argtypes = [vp, C.POINTER(IterInfo), C.c_int32]
        L.gem_nlr_buffer.argtypes = [vp, C.c_int32, C.POINTER(vp)]
        L.gem_nlr_path.argtypes = [vp]
        L.gem_nlr_path.restype = C.c_char_p
        L.gem_nlr_last_error.argtypes = [vp]
        L.gem_nlr_last_error.restype = C.c_char_p
        L.gem_nlr_destroy.argtypes = [vp]
        L.gem_nlr_host_job_device_bytes.argtypes = [pp]
        L.gem_nlr_host_job_device_bytes.restype = C.c_size_t
        L.gem_nlr_run_host.argtypes = [pp, vp, vp, vp, vp, C.c_size_t, vp, C.POINTER(C.c_double),
                                       C.POINTER(IterInfo), C.POINTER(C.c_int32)]
        L.gem_nlr_run_host_timed.argtypes = [pp, vp, vp, vp, vp, C.c_size_t, vp, C.POINTER(C.c_double),
                                             C.POINTER(IterInfo), C.POINTER(C.c_int32), C.POINTER(C.c_double)]
        L.gem_nlr_run_host_timed.restype = C.c_int
        L.gem_nlr_profile.argtypes = [vp, C.c_int32]
        L.gem_nlr_profile.restype = C.c_int
        L.gem_nlr_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.gem_nlr_profile_read.restype = C.c_int
        L.gem_nlr_launch_count.argtypes = [vp]
        L.gem_nlr_launch_count.restype = C.c_int64
        L.gem_nlr_selftest_wait_timeout.argtypes = [vp, C.c_uint32, C.POINTER(C.c_int64)]
        L.gem_nlr_selftest_wait_timeout.restype = C.c_int
        L.gem_nlr_column_sums_static.argtypes = [vp, C.c_int64, C.c_int32, vp, vp]
        L.gem_nlr_column_sums_static.restype = C.c_int
        L.gem_nlr_shard_exchange_bytes.argtypes = [pp, C.c_int32]
        L.gem_nlr_shard_exchange_bytes.restype = C.c_size_t
        L.gem_nlr_shard_attach.argtypes = [vp, C.c_int32, C.c_int32, C.c_int64, vp, vp, vp, vp, C.c_size_t]
        L.gem_nlr_shard_attach.restype = C.c_int
        L.gem_nlr_init_range.argtypes = [vp]
        L.gem_nlr_labels_spectral_scratch_bytes.argtypes = [pp]
        L.gem_nlr_labels_spectral_scratch_bytes.restype = C.c_size_t
        L.gem_nlr_labels_spectral.argtypes = [vp, vp, vp, C.c_size_t, C.c_int32, C.POINTER(C.c_int32)]
        L.gem_nlr_labels_spectral.restype = C.c_int
        for name in ("init_range", "create", "spectral_norm", "set_normalized", "step", "run", "labels", "objective",
                     "get_state", "set_state", "history", "buffer", "destroy", "run_host"):
            getattr(L, "gem_nlr_" + name).restype = C.c_int
        _lib = L
    return _lib


def make_params(n, d, K, r=None, alpha=0.1, beta=1.0, T=100, T_min=10, eps_d=0.01, eps_c=1e-4,
                center=1, x_inplace=1, pi_max_iters=100, pi_tol=1e-7, pi_seed=0, precision=-1,
                history=0) -> Params:
    return Params(int(n), int(d), int(K), int(r if r is not None else K), float(alpha), float(beta),
                  int(T), int(T_min), float(eps_d), float(eps_c), int(center), int(x_inplace),
                  int(pi_max_iters), float(pi_tol), int(pi_seed), int(precision), int(history))


def workspace_bytes(params: Params) -> int:
    return int(lib().gem_nlr_workspace_bytes(C.byref(params)))


def paper_storage_bytes(params: Params) -> int:
    return int(lib().gem_nlr_paper_storage_bytes(C.byref(params)))


def host_job_device_bytes(params: Params) -> int:
    return int(lib().gem_nlr_host_job_device_bytes(C.byref(params)))


class GemNlr:
    """One solver handle.  X and U are CUDA float32 tensors owned by the caller (U is updated in
    place); the workspace is a torch allocation kept alive by this object."""

    def __init__(self, X, U, K, stream=None, **kw):
        import torch
        assert X.is_cuda and U.is_cuda and X.dtype == torch.float32 and U.dtype == torch.float32
        assert X.is_contiguous() and U.is_contiguous() and X.shape[0] == U.shape[0]
        n, d = X.shape
        self.params = make_params(n, d, K, r=U.shape[1], **kw)
        self.X, self.U = X, U
        nbytes = workspace_bytes(self.params)
        if nbytes == 0:
            raise ValueError("invalid gem_nlr parameters")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=X.device)
        self._stream = stream if stream is not None else torch.cuda.current_stream(X.device)
        self._h = C.c_void_p()
        rc = lib().gem_nlr_create(C.byref(self._h), C.byref(self.params), X.data_ptr(), U.data_ptr(),
                                  self.workspace.data_ptr(), nbytes, self._stream.cuda_stream)
        if rc != OK:
            raise RuntimeError(f"gem_nlr_create failed: {rc}")

    # -- same names as the C entry points ---------------------------------------------------
    def spectral_norm(self) -> float:
        a = C.c_double()
        self._check(lib().gem_nlr_spectral_norm(self._h, C.byref(a)))
        return a.value

    def set_normalized(self, a: float = 1.0) -> None:
        self._check(lib().gem_nlr_set_normalized(self._h, float(a)))

    def init_range(self) -> int:
        """gem_nlr_init_range: U holds Z on entry, the data-informed starting factor on return."""
        return lib().gem_nlr_init_range(self._h)

    def step(self):
        info = IterInfo()
        rc = lib().gem_nlr_step(self._h, C.byref(info))
        return rc, info.as_dict()

    def run(self):
        info, iters = IterInfo(), C.c_int32()
        rc = lib().gem_nlr_run(self._h, C.byref(info), C.byref(iters))
        return rc, info.as_dict(), iters.value

    def labels(self, out=None):
        import torch
        if out is None:
            out = torch.empty(self.params.n, dtype=torch.int32, device=self.U.device)
        self._check(lib().gem_nlr_labels(self._h, out.data_ptr()))
        return out

    def labels_spectral(self, out=None, max_iter: int = 50):
        """gem_nlr_labels_spectral: (rc, labels, assignment passes); the scratch is a torch allocation."""
        import torch
        if out is None:
            out = torch.empty(self.params.n, dtype=torch.int32, device=self.U.device)
        nbytes = int(lib().gem_nlr_labels_spectral_scratch_bytes(C.byref(self.params)))
        scratch = torch.empty(nbytes, dtype=torch.uint8, device=self.U.device)
        passes = C.c_int32()
        rc = lib().gem_nlr_labels_spectral(self._h, out.data_ptr(), scratch.data_ptr(), nbytes, int(max_iter),
                                           C.byref(passes))
        return rc, out, passes.value

    def objective(self) -> float:
        f = C.c_double()
        self._check(lib().gem_nlr_objective(self._h, C.byref(f)))
        return f.value

    def get_state(self):
        import torch
        yt = torch.empty(self.params.n, dtype=torch.float32, device=self.U.device)
        t = C.c_int32()
        self._check(lib().gem_nlr_get_state(self._h, yt.data_ptr(), C.byref(t)))
        return yt, t.value

    def set_state(self, ytilde=None, t: int = 0) -> None:
        ptr = None if ytilde is None else ytilde.data_ptr()
        self._check(lib().gem_nlr_set_state(self._h, ptr, int(t)))

    def history(self, max_records: int):
        arr = (IterInfo * max_records)()
        n = lib().gem_nlr_history(self._h, arr, max_records)
        self._check(n)
        return [arr[i].as_dict() for i in range(n)]

    def buffer(self, which: int, numel: int, dtype=None):
        """A torch view of one of the workspace buffers (Theta, p, s, ytilde, ybar, X-hat)."""
        import torch
        ptr = C.c_void_p()
        self._check(lib().gem_nlr_buffer(self._h, which, C.byref(ptr)))
        off = ptr.value - self.workspace.data_ptr()
        if 0 <= off < self.workspace.numel():
            return self.workspace[off: off + 4 * numel].view(torch.float32)
        return self.X.view(-1)[:numel]

    def profile(self, enable: bool = True) -> None:
        self._check(lib().gem_nlr_profile(self._h, int(enable)))

    def profile_read(self):
        a, b, n = C.c_double(), C.c_double(), C.c_int64()
        self._check(lib().gem_nlr_profile_read(self._h, C.byref(a), C.byref(b), C.byref(n)))
        return a.value, b.value, n.value

    def selftest_wait_timeout(self, max_polls: int = 1024):
        """gem_nlr_selftest_wait_timeout: returns (rc, cycles of the wait that runs out, cycles of the wait after it)."""
        cyc = (C.c_int64 * 2)()
        rc = lib().gem_nlr_selftest_wait_timeout(self._h, int(max_polls), cyc)
        return rc, int(cyc[0]), int(cyc[1])

    def launch_count(self) -> int:
        return int(lib().gem_nlr_launch_count(self._h))

    def path(self) -> str:
        return lib().gem_nlr_path(self._h).decode()

    def last_error(self) -> str:
        return lib().gem_nlr_last_error(self._h).decode()

    def destroy(self) -> None:
        if self._h:
            lib().gem_nlr_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def _check(self, rc):
        if rc < 0:
            raise RuntimeError(f"gem_nlr call failed: {rc} {self.last_error()}")


def run_host(X_host, U_host, K, device_buffer, stream=None, want_labels=True, labels=None, phase_ms=None, **kw):
    """gem_nlr_run_host: numpy/pinned-torch host arrays in, U (in place) and labels out.  `labels` may be a
    caller-provided host array (n int32); `phase_ms`, a list, receives the five per-phase device times of
    gem_nlr_run_host_timed."""
    import numpy as np
    import torch
    n, d = X_host.shape
    params = make_params(n, d, K, r=U_host.shape[1], **kw)
    need = host_job_device_bytes(params)
    assert device_buffer.numel() * device_buffer.element_size() >= need
    st = stream if stream is not None else torch.cuda.current_stream(device_buffer.device)

    def ptr(x):
        return x.ctypes.data if isinstance(x, np.ndarray) else x.data_ptr()

    if want_labels and labels is None:
        labels = (np.empty(n, np.int32) if isinstance(X_host, np.ndarray)
                  else torch.empty(n, dtype=torch.int32, pin_memory=True))
    a, info, iters = C.c_double(), IterInfo(), C.c_int32()
    args = (C.byref(params), ptr(X_host), ptr(U_host), ptr(labels) if labels is not None else None,
            device_buffer.data_ptr(), device_buffer.numel() * device_buffer.element_size(),
            st.cuda_stream, C.byref(a), C.byref(info), C.byref(iters))
    if phase_ms is None:
        rc = lib().gem_nlr_run_host(*args)
    else:
        ph = (C.c_double * 5)()
        rc = lib().gem_nlr_run_host_timed(*args, ph)
        phase_ms[:] = list(ph)
    return rc, labels, a.value, info.as_dict(), iters.value


def column_sums_static(U, out=None, stream=None):
    """gem_nlr_column_sums_static: p = U^T 1 for a CUDA float32 matrix U, using only the scratch
    array built into the library -- for callers that cannot allocate device memory when they call
    (here `out` is allocated by torch only if the caller did not pass one).  Returns (rc, out);
    rc is E_TOO_LARGE when U has more than STATIC_MAX_R columns.  Does not synchronize."""
    import torch
    assert U.is_cuda and U.dtype == torch.float32 and U.is_contiguous() and U.dim() == 2
    n, r = U.shape
    if out is None:
        out = torch.empty(r, dtype=torch.float32, device=U.device)
    assert out.is_cuda and out.device == U.device and out.dtype == torch.float32 and out.numel() >= r
    st = stream if stream is not None else torch.cuda.current_stream(U.device)
    with torch.cuda.device(U.device):          # the entry point works on the current device
        rc = lib().gem_nlr_column_sums_static(U.data_ptr(), int(n), int(r), out.data_ptr(), st.cuda_stream)
    return rc, out
