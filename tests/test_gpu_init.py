"""GPU parity of the data-informed starting factor (gem_nlr_init_range) against its FP64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2609_36074_b200 as gem
from oracle import range_init
from gpu_helpers import make_solver, u_err

pytestmark = pytest.mark.gpu


def _problem(n, d, K, r, seed=0):
    spec = synth.MixtureSpec("t", n, d, K, "equal", 16.0, "unit", 10, seed)
    X, _, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    Z = np.random.default_rng([seed, 77]).standard_normal((n, r)).astype(np.float32)
    return Xhat, Z


# (n, d, K, r): ragged tiles in n, d and r; r > K as in the paper's own settings (r = 1.5 K .. 3 K); r <= d throughout
@pytest.mark.parametrize("n,d,K,r", [(2000, 16, 4, 4), (4099, 50, 20, 30), (4200, 64, 16, 48), (5000, 128, 16, 16),
                                     (20011, 32, 8, 8), (3000, 70, 20, 60)])
def test_init_range_matches_oracle(n, d, K, r):
    Xhat, Z = _problem(n, d, K, r)
    hp = synth.default_hparams(K)
    U0_ref, info = range_init.range_init(Xhat, Z, K)
    s = make_solver(Xhat, Z, K, hp)
    rc = s.init_range()
    assert rc == gem.OK, (rc, s.last_error())
    U0 = s.U.cpu().numpy()
    assert (U0 >= 0).all() and abs(float(np.sum(U0.astype(np.float64) ** 2)) - K) <= 1e-4 * K
    assert u_err(U0, U0_ref) <= 1e-4, u_err(U0, U0_ref)
    yt, t = s.get_state()
    assert t == 0 and float(yt.abs().max()) == 0.0
    # the iteration starts from it like from any caller-supplied factor
    st = oracle.State(Xhat, U0)
    for k in range(2):
        rc, inf = s.step()
        ref = st.step(K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], hp["T_min"])
        assert rc == gem.OK and inf["t"] == k and abs(inf["fhat"] - ref["fhat"]) <= 1e-5 * max(abs(ref["fhat"]), K / 100)
    assert u_err(s.U.cpu().numpy(), st.U) <= 1e-4
    s.destroy()


def test_init_range_rejects_rank_deficient_samples():
    Xhat, Z = _problem(3000, 24, 6, 6)
    hp = synth.default_hparams(6)
    # r > d: the sample cannot have full column rank
    Zw = np.random.default_rng(5).standard_normal((3000, 30)).astype(np.float32)
    s = make_solver(Xhat, Zw, 6, hp)
    assert s.init_range() == gem.E_INVALID
    s.destroy()
    # two equal columns of Z: M^T C M is singular, the factorization must stop with the breakdown code,
    # leave Z in place and the handle usable
    Zd = Z.copy()
    Zd[:, 3] = Zd[:, 1]
    s = make_solver(Xhat, Zd, 6, hp)
    assert s.init_range() == gem.E_BREAKDOWN
    assert np.array_equal(s.U.cpu().numpy(), Zd)
    s.U.copy_(torch.from_numpy(Z).cuda())
    assert s.init_range() == gem.OK
    U0_ref, _ = range_init.range_init(Xhat, Z, 6)
    assert u_err(s.U.cpu().numpy(), U0_ref) <= 1e-4
    s.destroy()
