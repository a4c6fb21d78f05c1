"""The failure path of the bounded device-side waits, exercised without faulting anything: a wait on a barrier that
nothing arrives on must run out, report GEM_NLR_E_TIMEOUT through the control block and return, leaving the context
usable."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2609_36074_b200 as gem
from gpu_helpers import make_solver, u_err

pytestmark = pytest.mark.gpu


def _problem():
    spec = synth.MixtureSpec("t", 5000, 32, 8, "equal", 16.0, "unit", 10, 0)
    X, _, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    return Xhat, synth.make_u0(spec.n, spec.K, spec.K), spec.K


def test_a_bounded_wait_runs_out_and_reports_timeout():
    Xhat, U0, K = _problem()
    hp = synth.default_hparams(K)
    s = make_solver(Xhat, U0, K, hp)
    assert s.path() == "ffma"                     # a family whose every stage hand-over is such a wait
    rc, info = s.step()
    assert rc == gem.OK
    rc, cyc_out, cyc_after = s.selftest_wait_timeout(1024)
    assert rc == gem.E_TIMEOUT                    # the wait gave up and said so; the kernel returned (we are here)
    assert cyc_out > 1024                         # it did poll max_polls times before giving up
    # with the abort flag up the next wait ends within 64 polls instead of the production limit of 2^20 (a poll may
    # suspend the thread for a hardware-chosen time, so the bound is on the poll count's order of magnitude)
    assert 0 < cyc_after < 2048 * (cyc_out / 1024) * 8
    # the handle now refuses to iterate, as after a real time-out ...
    rc2, _ = s.step()
    assert rc2 == gem.E_TIMEOUT
    # ... until the state is reloaded
    s.U.copy_(torch.from_numpy(U0).cuda())
    s.set_state(None, 0)
    rc3, info3 = s.step()
    assert rc3 == gem.OK and info3["t"] == 0
    s.destroy()
    # the context is intact: a fresh handle runs and agrees with the oracle
    f = make_solver(Xhat, U0, K, hp)
    st = oracle.State(Xhat, U0)
    for _ in range(3):
        rc, info = f.step()
        ref = st.step(K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], hp["T_min"])
        assert rc == gem.OK and info["dual_applied"] == ref["dual"]
    assert u_err(f.U.cpu().numpy(), st.U) <= 1e-4
    f.destroy()


def test_selftest_rejects_limits_that_could_spin_long():
    Xhat, U0, K = _problem()
    s = make_solver(Xhat, U0, K, synth.default_hparams(K))
    assert s.selftest_wait_timeout(0)[0] == gem.E_INVALID
    assert s.selftest_wait_timeout((1 << 20) + 1)[0] == gem.E_INVALID
    s.destroy()
