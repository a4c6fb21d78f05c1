"""Helpers shared by the GPU parity tests: build a solver on oracle-normalized data and compare."""
import numpy as np
import torch

import oracle
import paper_2609_36074_b200 as gem


def u_err(U_gpu: np.ndarray, U_ref: np.ndarray) -> float:
    """Scale-normalised max error: max |dU| / max |U_ref| (the pass/fail number for U)."""
    return float(np.abs(U_gpu.astype(np.float64) - U_ref.astype(np.float64)).max()
                 / max(np.abs(U_ref).max(), 1e-300))


def rel(a: float, b: float) -> float:
    return abs(a - b) / max(abs(b), 1e-300)


def make_solver(Xhat: np.ndarray, U0: np.ndarray, K: int, hp: dict, T: int = 100, **kw):
    """Solver whose X buffer already holds the oracle's X-hat (setup is tested separately)."""
    Xd = torch.from_numpy(np.ascontiguousarray(Xhat)).cuda()
    Ud = torch.from_numpy(np.ascontiguousarray(U0)).cuda()
    s = gem.GemNlr(Xd, Ud, K, alpha=hp["alpha"], beta=hp["beta"], eps_d=hp["eps_d"], eps_c=hp["eps_c"],
                   T=T, T_min=hp["T_min"], x_inplace=1, **kw)
    s.set_normalized(1.0)
    return s


def load_state(solver, U: np.ndarray, ytilde: np.ndarray, t: int):
    solver.U.copy_(torch.from_numpy(U))
    solver.set_state(torch.from_numpy(ytilde).cuda(), t)


def teacher_forced_steps(Xhat, U0, K, hp, steps, tol_u=1e-4, solver_kw=None, warm=0):
    """At each step both sides start from the oracle's (U_t, ytilde_t); returns per-step errors."""
    st = oracle.State(Xhat, U0)
    for _ in range(warm):
        st.step(K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], hp["T_min"])
    s = make_solver(Xhat, st.U, K, hp, T=10 ** 6, **(solver_kw or {}))
    out = []
    for _ in range(steps):
        load_state(s, st.U, st.ytilde, st.t)
        ref = st.step(K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], hp["T_min"])
        rc, info = s.step()
        assert rc >= 0, (rc, s.last_error())
        Ug = s.U.cpu().numpy()
        ytg, tg = s.get_state()
        rec = dict(u_err=u_err(Ug, st.U), a=rel(info["a"], ref["a"]), b=rel(info["b"], ref["b"]),
                   h=rel(info["h"], ref["h"]), c=rel(info["c"], ref["c"]),
                   delta=abs(info["delta_hat"] - ref["delta_hat"]), rho=rel(info["rho"], ref["rho"]),
                   fhat=rel(info["fhat"], ref["fhat"]), dual=(info["dual_applied"], ref["dual"]),
                   stop=(info["stop"], ref["stop"]),
                   yt=float(np.abs(ytg.cpu().numpy() - st.ytilde).max()), t=(tg, st.t), info=info, ref=ref)
        out.append(rec)
        assert rec["u_err"] <= tol_u, rec
    s.destroy()
    return out
