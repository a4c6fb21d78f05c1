"""GPU parity of the tcgen05 3xTF32 family (second product) against the CPU oracle."""
import numpy as np
import pytest

import oracle
import synth
import paper_2609_36074_b200 as gem
from gpu_helpers import make_solver, rel, teacher_forced_steps, u_err

pytestmark = pytest.mark.gpu
TOL_U, TOL_F = 1e-4, 1e-5


def _problem(n, d, K, seed=0):
    spec = synth.MixtureSpec("t", n, d, K, "equal", 16.0, "unit", 10, seed)
    X, lab, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    return Xhat, synth.make_u0(n, K, K, seed=seed)


# (n, d, r): one and several U panels, ragged last tile, more tiles than CTAs, r not a multiple of 16 or 32
TC_SHAPES = [(4000, 128, 16), (3001, 64, 100), (2500, 64, 16), (40003, 128, 16), (20011, 64, 100),
             (3000, 32, 8), (5000, 96, 36), (3000, 64, 160)]


@pytest.mark.parametrize("n,d,K", TC_SHAPES)
def test_tc_second_product_teacher_forced(n, d, K):
    Xhat, U0 = _problem(n, d, K)
    hp = synth.default_hparams(K)
    s = make_solver(Xhat, U0, K, hp, precision=1)
    assert "x3" in s.path(), s.path()          # TF32 or fp16 split, by shape
    s.destroy()
    recs = teacher_forced_steps(Xhat, U0, K, hp, steps=3, tol_u=TOL_U, solver_kw=dict(precision=1))
    for rec in recs:
        assert rec["a"] <= 1e-6 and rec["b"] <= 1e-6 and rec["h"] <= 1e-6, rec
        assert rec["c"] <= 2e-7 and rec["delta"] <= 1e-6, rec
        assert rec["rho"] <= 1e-5 and rec["fhat"] <= TOL_F, rec
        assert rec["dual"][0] == rec["dual"][1] and rec["stop"][0] == rec["stop"][1], rec


@pytest.mark.parametrize("n,d,K", [(9000, 128, 16), (6000, 64, 100)])
def test_tc_trajectory_matches_oracle_and_is_reproducible(n, d, K):
    Xhat, U0 = _problem(n, d, K)
    hp = dict(synth.default_hparams(K), eps_d=0.2)
    T = 30
    outs = []
    for _ in range(2):
        s = make_solver(Xhat, U0, K, hp, T=T, precision=1)
        rc, info, iters = s.run()
        assert rc == gem.ITER_CAP and iters == T, (rc, s.last_error())
        outs.append((s.U.cpu().numpy().copy(), info))
        s.destroy()
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]
    Uo, _, infoo, _, _ = oracle.run(Xhat, U0, K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], T, hp["T_min"])
    assert u_err(outs[0][0], Uo) <= TOL_U
    assert rel(outs[0][1]["rho"], infoo["rho"]) <= 1e-4


# ---- tiled tcgen05 kernels (wide d and r: 256-column blocks, d streamed in 32-feature chunks, fp16 split) ----
# one and several column blocks, r not a multiple of 16, ragged last row tile, more items than CTAs
# (4100, 1024, 48): a narrow factor whose resident Theta images do not fit in shared memory, so it takes the tiled kernels
TCG_SHAPES = [(4200, 64, 300), (4100, 768, 1000), (5000, 64, 520), (21000, 32, 260), (4200, 288, 600), (4100, 1024, 48),
              (19001, 288, 600), (40001, 64, 300)]


@pytest.mark.parametrize("n,d,K", TCG_SHAPES)
def test_tiled_tc_second_product_teacher_forced(n, d, K):
    Xhat, U0 = _problem(n, d, K)
    hp = synth.default_hparams(K)
    s = make_solver(Xhat, U0, K, hp, precision=1)
    assert "f16x3.tiled" in s.path(), s.path()
    s.destroy()
    recs = teacher_forced_steps(Xhat, U0, K, hp, steps=2, tol_u=TOL_U, solver_kw=dict(precision=1))
    for rec in recs:
        assert rec["a"] <= 1e-6 and rec["b"] <= 1e-6 and rec["h"] <= 1e-6, rec
        assert rec["c"] <= 2e-7 and rec["delta"] <= 1e-6, rec
        assert rec["rho"] <= 1e-5 and rec["fhat"] <= TOL_F, rec
        assert rec["dual"][0] == rec["dual"][1] and rec["stop"][0] == rec["stop"][1], rec


def test_tiled_tc_trajectory_is_reproducible_and_matches_oracle():
    n, d, K = 4400, 64, 300
    Xhat, U0 = _problem(n, d, K)
    hp = dict(synth.default_hparams(K), eps_d=0.2)
    T = 12
    outs = []
    for _ in range(2):
        s = make_solver(Xhat, U0, K, hp, T=T, precision=1)
        rc, info, iters = s.run()
        assert rc == gem.ITER_CAP and iters == T, (rc, s.last_error())
        outs.append((s.U.cpu().numpy().copy(), info))
        s.destroy()
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]
    Uo, _, infoo, _, _ = oracle.run(Xhat, U0, K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], T, hp["T_min"])
    assert u_err(outs[0][0], Uo) <= TOL_U
    assert rel(outs[0][1]["rho"], infoo["rho"]) <= 1e-4


def test_tiled_tc_trajectory_on_the_embedding_shape_twin():
    """Ten free-running iterations at d = 768, K = 1000 (the widest benchmark shape on n = 4100 rows, both
    products on the tiled kernels, the gate open from the start) against oracle.run."""
    n, d, K, T = 4100, 768, 1000, 10
    spec = synth.MixtureSpec("embedding-twin", n, d, K, "equal", -1.0, "sphere0.3", T, 0)
    X, _, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    U0 = synth.make_u0(n, K, K)
    hp = dict(synth.default_hparams(K), eps_d=0.5, T_min=4)
    s = make_solver(Xhat, U0, K, hp, T=T, precision=1, history=1)
    assert s.path() == "f16x3.tiled", s.path()
    rc, info, iters = s.run()
    assert rc == gem.ITER_CAP and iters == T, (rc, s.last_error())
    Ug = s.U.cpu().numpy()
    ytg = s.get_state()[0].cpu().numpy()
    hist = s.history(T)
    lab_g = s.labels().cpu().numpy()
    s.destroy()
    Uo, yto, infoo, _, _ = oracle.run(Xhat, U0, K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], T, hp["T_min"])
    assert u_err(Ug, Uo) <= TOL_U
    assert rel(info["fhat"], infoo["fhat"]) <= TOL_F and rel(info["rho"], infoo["rho"]) <= 1e-4
    assert sum(h["dual_applied"] for h in hist) > 0 and info["dual_applied"] == infoo["dual"]
    assert float(np.abs(ytg - yto).max()) <= 1e-4 * float(np.abs(yto).max()) + 1e-9
    lab_o = oracle.labels(Uo)
    diff = np.nonzero(lab_g != lab_o)[0]
    if diff.size:
        scale = float(np.abs(Uo).max())
        assert ((Uo[diff, lab_o[diff]].astype(np.float64) - Uo[diff, lab_g[diff]]) <= 2 * TOL_U * scale).all()
    assert diff.size <= 2


# ---- feature counts that are not a multiple of 32: the fp16-image kernels see d rounded up (zero features in the
# images, zero rows in Theta); includes the shapes of the paper's own scaling study (d = 50, r = 3 K) ----
# (n, d, K, r, kernel path)
PADDED_D_SHAPES = [(5000, 50, 60, 60, "f16x3"), (6001, 50, 20, 60, "f16x3"), (4500, 200, 100, 100, "f16x3.tiled"), (4400, 256, 128, 128, "f16x3.tiled"),
                   (4300, 300, 400, 400, "f16x3.tiled"), (4200, 110, 300, 300, "f16x3.tiled"),
                   (4300, 200, 100, 152, "f16x3.tiled"), (4200, 200, 100, 300, "f16x3.tiled")]


@pytest.mark.parametrize("n,d,K,r,path", PADDED_D_SHAPES)
def test_padded_feature_count_teacher_forced(n, d, K, r, path):
    spec = synth.MixtureSpec("t", n, d, K, "equal", 16.0, "unit", 10, 0)
    X, _, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    U0 = synth.make_u0(n, r, K, seed=0)
    hp = synth.default_hparams(K)
    s = make_solver(Xhat, U0, K, hp, precision=-1)
    assert s.path() == path, s.path()
    s.destroy()
    recs = teacher_forced_steps(Xhat, U0, K, hp, steps=3, tol_u=TOL_U, solver_kw=dict(precision=-1))
    for rec in recs:
        assert rec["a"] <= 1e-6 and rec["b"] <= 1e-6 and rec["h"] <= 1e-6, rec
        assert rec["c"] <= 2e-7 and rec["delta"] <= 1e-6, rec
        assert rec["rho"] <= 1e-5 and rec["fhat"] <= TOL_F, rec
        assert rec["dual"][0] == rec["dual"][1] and rec["stop"][0] == rec["stop"][1], rec


def test_padded_feature_count_full_run_with_setup():
    """Whole job on raw X (mean, power iteration, normalisation, images, iterations) at d = 50, r = 60."""
    import torch
    n, d, K, r, T = 20000, 50, 20, 60, 25
    spec = synth.MixtureSpec("t", n, d, K, "equal", 16.0, "unit", 10, 3)
    X, _, _ = synth.make_mixture(spec)
    U0 = synth.make_u0(n, r, K, seed=3)
    hp = dict(synth.default_hparams(K), eps_d=0.2)
    Xd, Ud = torch.from_numpy(X.copy()).cuda(), torch.from_numpy(U0.copy()).cuda()
    s = gem.GemNlr(Xd, Ud, K, alpha=hp["alpha"], beta=hp["beta"], eps_d=hp["eps_d"], eps_c=hp["eps_c"], T=T, T_min=T)
    a = s.spectral_norm()
    assert s.path() == "f16x3", s.path()
    rc, info, iters = s.run()
    assert rc == gem.ITER_CAP and iters == T, (rc, s.last_error())
    Xhat, a_o, _ = oracle.normalize(X)
    assert rel(a, a_o) <= 1e-5
    Uo, _, infoo, _, _ = oracle.run(Xhat, U0, K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], T, T)
    assert u_err(s.U.cpu().numpy(), Uo) <= 5e-4          # the two sides normalise with their own a (1e-5 apart)
    assert rel(info["fhat"], infoo["fhat"]) <= 1e-4 and rel(info["rho"], infoo["rho"]) <= 1e-3
    s.destroy()


# ---- x_inplace = 2: X-hat is given up after setup, the row-major fp16 images are built over it ----
@pytest.mark.parametrize("n,d,K,path", [(8200, 64, 100, "f16x3"), (4300, 288, 600, "f16x3.tiled"), (4200, 768, 1000, "f16x3.tiled"),
                                        (4500, 96, 36, "f16x3")])
def test_images_built_over_xhat_give_identical_iterates(n, d, K, path):
    import torch
    from paper_2609_36074_b200.binding import make_params
    spec = synth.MixtureSpec("t", n, d, K, "equal", 16.0, "unit", 10, 1)
    X, _, _ = synth.make_mixture(spec)
    U0 = synth.make_u0(n, K, K, seed=1)
    hp = dict(synth.default_hparams(K), eps_d=0.2)
    outs = []
    for mode in (1, 2):
        Xd, Ud = torch.from_numpy(X.copy()).cuda(), torch.from_numpy(U0.copy()).cuda()
        s = gem.GemNlr(Xd, Ud, K, alpha=hp["alpha"], beta=hp["beta"], eps_d=hp["eps_d"], eps_c=hp["eps_c"], T=6, T_min=2,
                       x_inplace=mode)
        assert s.path() == path, s.path()
        a = s.spectral_norm()
        rc, info, iters = s.run()
        assert rc >= 0 and iters == 6, (rc, s.last_error())
        outs.append((a, s.U.cpu().numpy().copy(), info, s.labels().cpu().numpy()))
        if mode == 2:
            with pytest.raises(RuntimeError):
                s.objective()                                   # reads X-hat itself: refused once it is given up
            assert s.init_range() == gem.E_INVALID
        s.destroy()
    assert outs[0][0] == outs[1][0] and outs[0][2] == outs[1][2]
    assert np.array_equal(outs[0][1], outs[1][1]) and np.array_equal(outs[0][3], outs[1][3])
    kw = dict(alpha=hp["alpha"], beta=hp["beta"], T=6, T_min=2)
    ws1 = gem.workspace_bytes(make_params(n, d, K, x_inplace=1, **kw))
    ws2 = gem.workspace_bytes(make_params(n, d, K, x_inplace=2, **kw))
    assert ws1 - ws2 >= 4 * n * d                               # the row-major pair no longer sits in the workspace


def test_giving_up_xhat_is_only_a_permission():
    """Shapes whose kernels still read X-hat keep it: x_inplace = 2 then behaves like 1."""
    import torch
    n, d, K = 5000, 32, 8                                       # FFMA family: no operand images at all
    spec = synth.MixtureSpec("t", n, d, K, "equal", 16.0, "unit", 10, 0)
    X, _, _ = synth.make_mixture(spec)
    U0 = synth.make_u0(n, K, K)
    hp = synth.default_hparams(K)
    Xd, Ud = torch.from_numpy(X.copy()).cuda(), torch.from_numpy(U0.copy()).cuda()
    s = gem.GemNlr(Xd, Ud, K, alpha=hp["alpha"], beta=hp["beta"], T=3, x_inplace=2)
    s.spectral_norm()
    f = s.objective()
    Xhat, _, _ = oracle.normalize(X)
    assert np.abs(Xd.cpu().numpy() - Xhat).max() <= 2e-6 * np.abs(Xhat).max()
    assert abs(f - oracle.objective(Xhat, U0, np.zeros(n, np.float32), hp["beta"])) <= 1e-5 * abs(f)
    s.destroy()
