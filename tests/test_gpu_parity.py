"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs."""
import dataclasses
import itertools

import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2609_36074_b200 as gem
from gpu_helpers import load_state, make_solver, rel, teacher_forced_steps, u_err

pytestmark = pytest.mark.gpu

# per-step tolerances (fp32 path): U scale-normalised max error 1e-4, objective 1e-5 relative
TOL_U, TOL_F = 1e-4, 1e-5


def _problem(n, d, K, r=None, seed=0, centre_var=25.0):
    spec = synth.MixtureSpec("t", n, d, K, "equal", centre_var, "unit", 10, seed)
    X, lab, _ = synth.make_mixture(spec)
    Xhat, a, mean = oracle.normalize(X)
    U0 = synth.make_u0(n, r or K, K, seed=seed)
    return X, lab, Xhat, U0


# shapes span several tiles and ragged tails in n, d and r (64-wide tiles on the generic path)
SHAPES = [(2000, 16, 4, None), (1000, 3, 3, None), (4099, 50, 20, 30), (777, 70, 100, None),
          (3001, 130, 5, 67), (12, 3, 2, None)]


@pytest.mark.parametrize("n,d,K,r", SHAPES)
def test_teacher_forced_steps_match_oracle(n, d, K, r):
    _, _, Xhat, U0 = _problem(n, d, K, r)
    hp = synth.default_hparams(K)
    recs = teacher_forced_steps(Xhat, U0, K, hp, steps=4, tol_u=TOL_U)
    for rec in recs:
        assert rec["a"] <= 1e-6 and rec["b"] <= 1e-6 and rec["h"] <= 1e-6, rec
        assert rec["c"] <= 2e-7 and rec["delta"] <= 1e-6, rec
        assert rec["rho"] <= 1e-5 and rec["fhat"] <= TOL_F, rec
        assert rec["dual"][0] == rec["dual"][1] and rec["stop"][0] == rec["stop"][1], rec
        assert rec["yt"] <= 1e-9 and rec["t"][0] == rec["t"][1], rec


def test_teacher_forced_steps_near_convergence_with_dual_updates():
    """Late iterations of config 1: the gate fires, ytilde moves, the clamp is active on most entries."""
    spec = synth.config(1)
    X, _, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    hp = synth.default_hparams(spec.K)
    recs = teacher_forced_steps(Xhat, synth.make_u0(spec.n, spec.K, spec.K), spec.K, hp, steps=6, warm=150)
    assert any(r["dual"][1] for r in recs)
    for rec in recs:
        assert rec["dual"][0] == rec["dual"][1]
        assert rec["fhat"] <= TOL_F and rec["rho"] <= 1e-4 and rec["yt"] <= 1e-9, rec


def test_config1_trajectory_and_labels():
    """Free-running config 1 (tiny mixture): same gates, same stop iteration, U within tolerance,
    argmax labels bit-exact against the oracle and equal to the planted partition."""
    spec = synth.config(1)
    X, lab, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    hp = synth.default_hparams(spec.K)
    U0 = synth.make_u0(spec.n, spec.K, spec.K)
    # the configured 200 iterations
    s = make_solver(Xhat, U0, spec.K, hp, T=spec.iters, history=1)
    rc, info, iters = s.run()
    Uo, yto, infoo, iterso, rco = oracle.run(Xhat, U0, spec.K, hp["alpha"], hp["beta"], hp["eps_d"],
                                             hp["eps_c"], spec.iters, hp["T_min"])
    assert rc == gem.ITER_CAP and iters == iterso == spec.iters
    assert u_err(s.U.cpu().numpy(), Uo) <= TOL_U
    assert rel(info["fhat"], infoo["fhat"]) <= TOL_F
    hist = s.history(spec.iters)
    assert len(hist) == spec.iters and [h["t"] for h in hist] == list(range(spec.iters))
    st = oracle.State(Xhat, U0)
    for hrec in hist:
        ref = st.step(spec.K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], hp["T_min"])
        assert hrec["dual_applied"] == ref["dual"], hrec
        # the objective crosses zero along this trajectory: its terms are O(K), so the relative
        # tolerance is taken against max(|f|, K / 100)
        assert abs(hrec["fhat"] - ref["fhat"]) <= TOL_F * max(abs(ref["fhat"]), 0.01 * spec.K), hrec
        assert abs(hrec["delta_hat"] - ref["delta_hat"]) <= 1e-6
    # run on to convergence
    s.destroy()
    s = make_solver(Xhat, U0, spec.K, hp, T=1000)
    rc, info, iters = s.run()
    Uo, _, infoo, iterso, _ = oracle.run(Xhat, U0, spec.K, hp["alpha"], hp["beta"], hp["eps_d"],
                                         hp["eps_c"], 1000, hp["T_min"])
    assert rc == gem.CONVERGED and info["stop"] == 1 and abs(iters - iterso) <= 1
    assert u_err(s.U.cpu().numpy(), Uo) <= 5e-4          # stop may differ by one iteration at the threshold
    pred = s.labels().cpu().numpy()
    assert np.array_equal(pred, oracle.labels(Uo))
    best = max(np.mean(np.array(perm)[pred] == lab) for perm in itertools.permutations(range(spec.K)))
    assert best == 1.0
    assert rel(s.objective(), oracle.objective(Xhat, s.U.cpu().numpy(), s.get_state()[0].cpu().numpy(),
                                               hp["beta"])) <= TOL_F
    s.destroy()


def _same_partition(a, b):
    pairs = set(zip(a.tolist(), b.tolist()))
    return len(pairs) == len(set(a.tolist())) == len(set(b.tolist()))


@pytest.mark.parametrize("K,seed", [(2, 0), (2, 1), (3, 0), (3, 1), (3, 2)])
def test_tiny_mixtures_recover_exact_kmeans_partition(K, seed):
    """n = 12 well-separated points: the planted partition is the brute-force optimum (checked in the
    oracle's own tests); the GPU solver must return it."""
    X, planted = synth.separated_tiny_mixture(12, K, seed=seed)
    U0 = synth.make_u0(12, K, K, seed=seed)
    Xd, Ud = torch.from_numpy(X).cuda(), torch.from_numpy(U0).cuda()
    s = gem.GemNlr(Xd, Ud, K, alpha=0.1, beta=1.0, eps_d=0.05, eps_c=1e-4, T=5000, T_min=10)
    a = s.spectral_norm()
    a_ref, _ = oracle.spectral_norm(X)
    assert rel(a, a_ref) <= 1e-5
    rc, info, iters = s.run()
    assert rc == gem.CONVERGED and iters < 5000
    pred = s.labels().cpu().numpy()
    assert _same_partition(pred, planted)
    Xhat, _, _ = oracle.normalize(X)
    Uo, _, _, _, _ = oracle.run(Xhat, U0, K, 0.1, 1.0, 0.05, 1e-4, 5000, 10)
    assert np.array_equal(pred, oracle.labels(Uo))
    s.destroy()


@pytest.mark.parametrize("n,d,center", [(5000, 16, 1), (3000, 37, 1), (2048, 128, 0), (700, 300, 1), (1500, 768, 1), (900, 512, 0)])
def test_setup_matches_oracle(n, d, center):
    rng = np.random.default_rng(n + d)
    X = (rng.standard_normal((n, d)) * rng.uniform(0.3, 3.0, size=d) + rng.uniform(-4, 4, size=d)
         + 2.0 * rng.integers(0, 3, size=(n, 1))).astype(np.float32)
    a_ref, mean = oracle.spectral_norm(X, bool(center))
    Xhat_ref = np.empty_like(X)
    oracle.lib().nlr_oracle_normalize(X, n, d, mean, a_ref, Xhat_ref)
    for inplace in (1, 0):
        Xd = torch.from_numpy(X).cuda()
        Ud = torch.from_numpy(synth.make_u0(n, 3, 3)).cuda()
        s = gem.GemNlr(Xd, Ud, 3, center=center, x_inplace=inplace, pi_max_iters=300, pi_tol=1e-10)
        a = s.spectral_norm()
        assert a <= a_ref * (1 + 1e-9) and rel(a, a_ref) <= 1e-5, (a, a_ref)
        Xh = s.buffer(5, n * d).cpu().numpy().reshape(n, d)
        assert np.abs(Xh - Xhat_ref).max() <= 2e-5 * np.abs(Xhat_ref).max()
        if not inplace:
            assert np.array_equal(Xd.cpu().numpy(), X)     # the caller's X is left alone
        s.destroy()


def test_breakdown_status_and_unscaled_factor():
    X, _ = synth.separated_tiny_mixture(9, 3, seed=0)
    Xhat, _, _ = oracle.normalize(X)
    hp = dict(alpha=50.0, beta=1.0, eps_d=0.05, eps_c=1e-4, T_min=10)
    s = make_solver(Xhat, synth.make_u0(9, 3, 3), 3, hp, T=50)
    rc, info = s.step()
    assert rc == gem.E_BREAKDOWN and info["status"] == gem.E_BREAKDOWN and info["a"] == 0.0
    assert (s.U.cpu().numpy() == 0).all()
    assert s.step()[0] == gem.E_BREAKDOWN        # sticky until a new state is loaded
    s.destroy()
    s = make_solver(Xhat, synth.make_u0(9, 3, 3), 3, hp, T=50)
    rc, info, iters = s.run()
    assert rc == gem.E_BREAKDOWN and iters == 0
    s.destroy()


def test_nonfinite_input_is_reported():
    """A NaN in U reaches b = ||U||_F^2 and is reported as non-finite.  A NaN in X makes every
    tentative entry NaN, which max(., 0) maps to 0, so W vanishes: breakdown -- on both sides."""
    _, _, Xhat, U0 = _problem(500, 8, 3)
    hp = synth.default_hparams(3)
    Ubad = U0.copy()
    Ubad[17, 1] = np.nan
    s = make_solver(Xhat, Ubad, 3, hp)
    rc, info = s.step()
    assert rc == gem.E_NONFINITE and info["status"] == gem.E_NONFINITE
    s.destroy()
    assert oracle.State(Xhat, Ubad).step(3, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 10)["status"] == -5
    Xbad = Xhat.copy()
    Xbad[17, 3] = np.nan
    s = make_solver(Xbad, U0, 3, hp)
    rc, info = s.step()
    assert rc == gem.E_BREAKDOWN
    s.destroy()
    assert oracle.State(Xbad, U0).step(3, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 10)["status"] == -4


def test_argument_errors():
    import ctypes as C
    from paper_2609_36074_b200.binding import make_params
    L = gem.lib()
    X = torch.zeros(64, 8, device="cuda")
    U = torch.zeros(64, 4, device="cuda")
    P = make_params(64, 8, 4)
    ws = torch.empty(gem.workspace_bytes(P), dtype=torch.uint8, device="cuda")
    h = C.c_void_p()
    assert L.gem_nlr_create(C.byref(h), C.byref(P), X.data_ptr(), U.data_ptr(), ws.data_ptr(), 16, None) == gem.E_WORKSPACE
    assert L.gem_nlr_create(C.byref(h), C.byref(P), None, U.data_ptr(), ws.data_ptr(), ws.numel(), None) == gem.E_INVALID
    assert L.gem_nlr_create(C.byref(h), C.byref(P), X.data_ptr() + 4, U.data_ptr(), ws.data_ptr(), ws.numel(), None) == gem.E_INVALID
    bad = make_params(64, 8, 4, r=2)
    assert L.gem_nlr_create(C.byref(h), C.byref(bad), X.data_ptr(), U.data_ptr(), ws.data_ptr(), ws.numel(), None) == gem.E_INVALID
    assert L.gem_nlr_create(C.byref(h), C.byref(P), X.data_ptr(), U.data_ptr(), ws.data_ptr(), ws.numel(), None) == gem.OK
    assert L.gem_nlr_step(h, None) == gem.E_NOT_READY
    assert L.gem_nlr_destroy(h) == gem.OK


def test_runs_are_bitwise_reproducible_and_steps_equal_run():
    _, _, Xhat, U0 = _problem(3000, 24, 6)
    hp = synth.default_hparams(6)
    outs = []
    for _ in range(2):
        s = make_solver(Xhat, U0, 6, hp, T=25)
        rc, info, iters = s.run()
        outs.append((s.U.cpu().numpy().copy(), s.get_state()[0].cpu().numpy().copy(), info))
        s.destroy()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    assert outs[0][2] == outs[1][2]
    s = make_solver(Xhat, U0, 6, hp, T=25)
    for _ in range(25):
        rc, info = s.step()
    assert u_err(s.U.cpu().numpy(), outs[0][0]) <= 1e-5
    assert rel(info["rho"], outs[0][2]["rho"]) <= 1e-5
    s.destroy()


def test_labels_tie_break_and_wide_rows():
    U = np.zeros((70, 40), np.float32)
    rng = np.random.default_rng(0)
    U[:] = rng.integers(0, 4, size=U.shape).astype(np.float32)      # many ties
    U[5] = 0.0
    for r in (40, 7):
        Ur = np.ascontiguousarray(U[:, :r])
        Xd = torch.zeros(70, 4, device="cuda")
        s = gem.GemNlr(Xd, torch.from_numpy(Ur).cuda(), 2)
        assert np.array_equal(s.labels().cpu().numpy(), oracle.labels(Ur))
        s.destroy()
    # every read-out kernel (thread per row with 16-byte loads; warp per 8 / 4 / 2 / 1 rows; the scalar fallback),
    # ragged row counts, many ties
    for n, r in ((1003, 16), (1003, 32), (517, 100), (1001, 128), (301, 200), (203, 300), (77, 1000), (50, 1030)):
        Ur = rng.integers(0, 3, size=(n, r)).astype(np.float32)
        Ur[n // 2] = 1.0
        Xd = torch.zeros(n, 4, device="cuda")
        s = gem.GemNlr(Xd, torch.from_numpy(Ur).cuda(), 2)
        assert np.array_equal(s.labels().cpu().numpy(), oracle.labels(Ur)), (n, r)
        s.destroy()


def test_host_buffer_job_matches_device_job():
    spec = synth.config(1).with_n(1500)
    X, lab, _ = synth.make_mixture(spec)
    hp = synth.default_hparams(spec.K)
    U0 = synth.make_u0(spec.n, spec.K, spec.K)
    kw = dict(alpha=hp["alpha"], beta=hp["beta"], eps_d=hp["eps_d"], eps_c=hp["eps_c"], T=40, T_min=hp["T_min"])
    Xd, Ud = torch.from_numpy(X).cuda(), torch.from_numpy(U0).cuda()
    s = gem.GemNlr(Xd, Ud, spec.K, **kw)
    a = s.spectral_norm()
    rc, info, iters = s.run()
    lab_dev = s.labels().cpu().numpy()
    from paper_2609_36074_b200.binding import make_params
    P = make_params(spec.n, spec.d, spec.K, **kw)
    buf = torch.empty(gem.host_job_device_bytes(P), dtype=torch.uint8, device="cuda")
    Uh = U0.copy()
    rc2, lab_host, a2, info2, iters2 = gem.run_host(X, Uh, spec.K, buf, **kw)
    assert (rc2, iters2, a2) == (rc, iters, a) and info2 == info
    assert np.array_equal(Uh, s.U.cpu().numpy()) and np.array_equal(lab_host, lab_dev)
    s.destroy()


# ---- TMA-staged FFMA family (skinny shapes) ------------------------------------------------------
# n spans many 64..256-row tiles, more tiles than CTAs in one case, and a ragged last tile
FFMA_SHAPES = [(5000, 32, 8), (3333, 128, 16), (2500, 64, 16), (4097, 64, 8), (3001, 32, 16),
               (60001, 32, 8), (40003, 128, 16)]


@pytest.mark.parametrize("n,d,K", FFMA_SHAPES)
def test_ffma_family_teacher_forced(n, d, K):
    _, _, Xhat, U0 = _problem(n, d, K)
    hp = synth.default_hparams(K)
    s = make_solver(Xhat, U0, K, hp, precision=0)
    assert s.path() == "ffma"
    s.destroy()
    recs = teacher_forced_steps(Xhat, U0, K, hp, steps=3, tol_u=TOL_U, solver_kw=dict(precision=0))
    _check_recs(recs)


def _check_recs(recs):
    for rec in recs:
        assert rec["a"] <= 1e-6 and rec["b"] <= 1e-6 and rec["h"] <= 1e-6, rec
        assert rec["c"] <= 2e-7 and rec["delta"] <= 1e-6, rec
        assert rec["rho"] <= 1e-5 and rec["fhat"] <= TOL_F, rec
        assert rec["dual"][0] == rec["dual"][1] and rec["stop"][0] == rec["stop"][1], rec
        assert rec["yt"] <= 1e-9, rec


# ---- warp-level tensor-core kernels of the same family (mma.sync TF32, 3-product split) ----------
MMA_SHAPES = [(3333, 128, 16), (2500, 64, 16), (4097, 64, 8), (1024, 128, 8), (40003, 128, 16), (50001, 64, 16)]


@pytest.mark.parametrize("n,d,K", MMA_SHAPES)
def test_mma_family_teacher_forced(n, d, K):
    _, _, Xhat, U0 = _problem(n, d, K)
    hp = synth.default_hparams(K)
    s = make_solver(Xhat, U0, K, hp)          # automatic selection takes these kernels for d >= 64
    assert s.path() == "mma.tf32x3"
    s.destroy()
    _check_recs(teacher_forced_steps(Xhat, U0, K, hp, steps=3, tol_u=TOL_U, solver_kw=dict(precision=3)))


# wide factors: r in N tiles of 8 columns, the last one partly filled (r = 100, 60) or full (104, 64)
MMAW_SHAPES = [(3000, 64, 100), (2050, 64, 64), (5000, 32, 104), (3001, 64, 60), (30011, 64, 100)]


@pytest.mark.parametrize("n,d,K", MMAW_SHAPES)
def test_mma_wide_family_teacher_forced(n, d, K):
    _, _, Xhat, U0 = _problem(n, d, K)
    hp = synth.default_hparams(K)
    s = make_solver(Xhat, U0, K, hp, precision=3)
    assert s.path() == "mma.tf32x3"
    s.destroy()
    _check_recs(teacher_forced_steps(Xhat, U0, K, hp, steps=3, tol_u=TOL_U, solver_kw=dict(precision=3)))


@pytest.mark.parametrize("n,d,K", [(9000, 128, 16), (12000, 64, 8), (8000, 64, 100)])
def test_mma_family_trajectory_matches_oracle(n, d, K):
    _, _, Xhat, U0 = _problem(n, d, K)
    hp = dict(synth.default_hparams(K), eps_d=0.2)
    T = 40
    outs = []
    for _ in range(2):
        s = make_solver(Xhat, U0, K, hp, T=T, precision=3, history=1)
        assert s.path() == "mma.tf32x3"
        rc, info, iters = s.run()
        assert rc == gem.ITER_CAP and iters == T
        outs.append((s.U.cpu().numpy().copy(), s.get_state()[0].cpu().numpy().copy(), info, s.history(T)))
        s.destroy()
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][2] == outs[1][2]
    Uo, yto, infoo, iterso, _ = oracle.run(Xhat, U0, K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"],
                                           T, hp["T_min"])
    U, yt, info, hist = outs[0]
    assert any(h["dual_applied"] for h in hist)
    assert u_err(U, Uo) <= TOL_U
    assert np.abs(yt - yto).max() <= 1e-4 * max(np.abs(yto).max(), 1e-30)
    assert rel(info["rho"], infoo["rho"]) <= 1e-4 and abs(info["delta_hat"] - infoo["delta_hat"]) <= 1e-6


@pytest.mark.parametrize("n,d,K", [(20000, 32, 8), (9000, 128, 16)])
def test_ffma_family_trajectory_matches_generic_and_oracle(n, d, K):
    """40 free-running iterations with an eager dual gate: specialised kernels against the generic
    family on the GPU and against the oracle; two runs are bitwise equal."""
    _, _, Xhat, U0 = _problem(n, d, K)
    hp = dict(synth.default_hparams(K), eps_d=0.2)
    T = 40
    outs = {}
    for name, prec in (("ffma", 0), ("ffma2", 0), ("generic", 2)):
        s = make_solver(Xhat, U0, K, hp, T=T, precision=prec, history=1)
        assert s.path() == ("generic" if prec == 2 else "ffma")
        rc, info, iters = s.run()
        assert rc == gem.ITER_CAP and iters == T
        outs[name] = (s.U.cpu().numpy().copy(), s.get_state()[0].cpu().numpy().copy(), info, s.history(T))
        s.destroy()
    assert np.array_equal(outs["ffma"][0], outs["ffma2"][0]) and outs["ffma"][2] == outs["ffma2"][2]
    Uo, yto, infoo, iterso, _ = oracle.run(Xhat, U0, K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"],
                                           T, hp["T_min"])
    assert any(h["dual_applied"] for h in outs["ffma"][3])
    for name in ("ffma", "generic"):
        U, yt, info, hist = outs[name]
        assert u_err(U, Uo) <= TOL_U, name
        assert np.abs(yt - yto).max() <= 1e-4 * max(np.abs(yto).max(), 1e-30), name
        assert rel(info["rho"], infoo["rho"]) <= 1e-4 and abs(info["delta_hat"] - infoo["delta_hat"]) <= 1e-6
    assert [h["dual_applied"] for h in outs["ffma"][3]] == [h["dual_applied"] for h in outs["generic"][3]]
