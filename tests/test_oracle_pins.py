"""Pins for the CPU oracle: each test checks it against something other than itself
(a definition written with explicit n x n matrices, finite differences, a closed
form, a library routine, brute force)."""
import dataclasses
import itertools

import numpy as np
import pytest

import oracle
import synth


def _small_problem(n=40, d=5, r=3, seed=0, positive_margin=False):
    rng = np.random.default_rng(seed)
    X = (rng.standard_normal((n, d)) + 3.0 * rng.integers(0, 3, size=(n, 1))).astype(np.float32)
    Xhat, a, mean = oracle.normalize(X)
    U = synth.make_u0(n, r, r, seed=seed)
    if positive_margin:
        U = (0.5 * U + 0.5 * np.sqrt(r / (n * r))).astype(np.float32)
        U *= np.float32(np.sqrt(r / np.sum(U.astype(np.float64) ** 2)))
    yt = (0.01 * rng.standard_normal(n)).astype(np.float32)
    return X, Xhat, a, U, yt


def _objective_definition(Xhat, U, ytilde, beta):
    """Eq. "normalized" with the explicit n x n matrices, in fp64."""
    Xh = Xhat.astype(np.float64)
    U = U.astype(np.float64)
    n = U.shape[0]
    A_hat = -Xh @ Xh.T
    Z = U @ U.T
    y = np.sqrt(n) * ytilde.astype(np.float64)
    h = (Z @ np.ones(n) - np.ones(n)) / np.sqrt(n)
    return np.sum(A_hat * Z) + y @ h + 0.5 * beta * (h @ h)


def test_objective_matches_definition():
    _, Xhat, _, U, yt = _small_problem()
    for beta in (0.5, 1.0, 3.0):
        ref = _objective_definition(Xhat, U, yt, beta)
        got = oracle.objective(Xhat, U, yt, beta)
        assert abs(got - ref) <= 1e-12 * max(1.0, abs(ref))


def test_residual_and_theta_match_library_products():
    _, Xhat, _, U, _ = _small_problem(n=57, d=7, r=4, seed=3)
    p, q = oracle.residual(U)
    U64 = U.astype(np.float64)
    np.testing.assert_allclose(p, U64.sum(0), rtol=1e-7)
    np.testing.assert_allclose(q, U64 @ p.astype(np.float64) - 1.0, atol=1e-7)
    np.testing.assert_allclose(oracle.theta(Xhat, U), Xhat.astype(np.float64).T @ U64,
                               rtol=1e-6, atol=1e-9)


def test_gradient_step_matches_finite_differences():
    """With a tiny step and a strictly positive U no entry is clamped, so
    W = U - alpha * grad and the gradient can be read back from one step."""
    _, Xhat, _, U, yt = _small_problem(positive_margin=True)
    n, r = U.shape
    alpha, beta = 1e-2, 1.0
    st = oracle.State(Xhat, U, yt)
    info = st.step(K=r, alpha=alpha, beta=beta, eps_d=0.0, eps_c=0.0, T_min=1)
    assert info["status"] == 0 and info["dual"] == 0
    W = st.U.astype(np.float64) / info["c"]
    assert (W > 0).all()
    grad_from_step = (U.astype(np.float64) - W) / alpha
    rng = np.random.default_rng(1)
    eps = 1e-3
    for _ in range(12):
        i, j = rng.integers(n), rng.integers(r)
        Up, Um = U.copy(), U.copy()
        Up[i, j] += np.float32(eps)
        Um[i, j] -= np.float32(eps)
        hstep = float(Up[i, j]) - float(Um[i, j])
        fd = (oracle.objective(Xhat, Up, yt, beta) - oracle.objective(Xhat, Um, yt, beta)) / hstep
        assert abs(fd - grad_from_step[i, j]) <= 2e-5 * max(1.0, abs(fd)), (i, j, fd, grad_from_step[i, j])


def test_gradient_formula_explicit():
    """Eq. "gradient": 2 A-hat U + ybar (U^T 1)^T + 1 (U^T ybar)^T with explicit matrices."""
    _, Xhat, _, U, yt = _small_problem(positive_margin=True, seed=5)
    n, r = U.shape
    alpha, beta = 5e-3, 2.0
    Xh, U64 = Xhat.astype(np.float64), U.astype(np.float64)
    one = np.ones(n)
    g = U64 @ (U64.T @ one) - one
    ybar = yt.astype(np.float64) + (beta / n) * g
    grad = 2.0 * (-(Xh @ Xh.T)) @ U64 + np.outer(ybar, U64.T @ one) + np.outer(one, U64.T @ ybar)
    st = oracle.State(Xhat, U, yt)
    info = st.step(K=r, alpha=alpha, beta=beta, eps_d=0.0, eps_c=0.0, T_min=1)
    W = st.U.astype(np.float64) / info["c"]
    np.testing.assert_allclose((U64 - W) / alpha, grad, atol=3e-5)


def _alm_unnormalized_step(Xc, U, y, alpha, beta, K):
    """One primal step (S = 1, no trace multiplier) of the unnormalized augmented-Lagrangian
    method on A = -Xc Xc^T, then the residual used by its dual ascent."""
    n = U.shape[0]
    one = np.ones(n)
    A = -(Xc @ Xc.T)
    ybar = y + beta * (U @ (U.T @ one) - one)
    grad = (2.0 * A + np.outer(one, ybar) + np.outer(ybar, one)) @ U
    V = np.maximum(U - alpha * grad, 0.0)
    Unew = np.sqrt(K) * V / np.linalg.norm(V)
    s = Unew @ (Unew.T @ one) - one
    return Unew, s


def test_normalized_step_equals_unnormalized_alm_step():
    """Spectral normalization is a reparametrization: a step with (alpha, beta, y) on X-hat is a
    step of the unnormalized method on the centered data with alpha/a^2, a^2 beta/n, a^2 y/sqrt(n)."""
    X, Xhat, a, U, yt = _small_problem(n=30, d=4, r=3, seed=2)
    n, r = U.shape
    alpha, beta = 0.05, 1.5
    # use the rounded X-hat so both sides see the same data: Xc := a * Xhat
    Xc = a * Xhat.astype(np.float64)
    Uref, s = _alm_unnormalized_step(Xc, U.astype(np.float64), a * a * yt.astype(np.float64),
                                     alpha / (a * a), a * a * beta / n, r)
    st = oracle.State(Xhat, U, yt)
    info = st.step(K=r, alpha=alpha, beta=beta, eps_d=1e9, eps_c=0.0, T_min=1)  # gate always fires
    assert info["dual"] == 1
    np.testing.assert_allclose(st.U, Uref, atol=2e-7)
    y_unnorm = a * a * yt.astype(np.float64) + (a * a * beta / n) * s
    np.testing.assert_allclose(a * a * st.ytilde.astype(np.float64), y_unnorm,
                               atol=1e-6 * max(1.0, np.abs(y_unnorm).max()))


def test_movement_identity_matches_direct_norm():
    _, Xhat, _, U, yt = _small_problem(n=200, d=6, r=4, seed=7)
    st = oracle.State(Xhat, U, yt)
    for _ in range(5):
        Uprev = st.U.astype(np.float64).copy()
        info = st.step(K=4, alpha=0.05, beta=1.0, eps_d=0.01, eps_c=1e-4, T_min=1)
        direct = np.linalg.norm(st.U.astype(np.float64) - Uprev) / np.sqrt(4)
        assert abs(info["delta_hat"] - direct) <= 1e-6
        # statistics themselves
        assert abs(info["b"] - np.sum(Uprev ** 2)) <= 1e-12 * info["b"]
        W = st.U.astype(np.float64) / info["c"]
        assert abs(info["a"] - np.sum(W ** 2)) <= 1e-6 * info["a"]
        assert abs(info["h"] - np.sum(W * Uprev)) <= 1e-6 * abs(info["h"])
        assert abs(info["c"] - float(np.float32(np.sqrt(4 / info["a"])))) <= 2e-7 * info["c"]
        # Section 4.3: rho = ||q||_2 / sqrt(n), with q = U p - 1 taken from the NEW factor
        Unew = st.U.astype(np.float64)
        q_direct = Unew @ Unew.sum(0) - 1.0
        rho_direct = np.linalg.norm(q_direct) / np.sqrt(200)
        assert abs(info["rho"] - rho_direct) <= 1e-6 * rho_direct
        assert abs(info["rho"] - np.linalg.norm(st.q.astype(np.float64)) / np.sqrt(200)) <= 1e-12 * info["rho"]


def _trajectory_with_gate_crossing(eps_d, eps_c, T_min, iters=400):
    spec = dataclasses.replace(synth.config(1).with_n(400), seed=1)
    X, _, _ = synth.make_mixture(spec)
    hp = synth.default_hparams(spec.K)
    Xhat, _, _ = oracle.normalize(X)
    st = oracle.State(Xhat, synth.make_u0(spec.n, spec.K, spec.K, seed=1))
    out = []
    for t in range(iters):
        Uprev = st.U.astype(np.float64).copy()
        yprev = st.ytilde.copy()
        info = st.step(spec.K, hp["alpha"], hp["beta"], eps_d, eps_c, T_min)
        assert info["status"] == 0 and info["t"] == t
        direct = np.linalg.norm(st.U.astype(np.float64) - Uprev) / np.sqrt(spec.K)
        out.append((t, info, direct, not np.array_equal(yprev, st.ytilde)))
        if info["stop"]:
            break
    return out


def test_dual_gate_is_the_main_text_test_on_the_movement():
    """Section 4.3: the dual ascent fires exactly when delta-hat < eps_d. The comparison is made
    here on delta-hat itself (and on the directly computed movement), not on the squared form the
    oracle evaluates, over a trajectory that crosses the threshold."""
    eps_d = 0.05
    traj = _trajectory_with_gate_crossing(eps_d, eps_c=1e-4, T_min=10)
    seen = set()
    for t, info, direct, y_changed in traj:
        if abs(direct - eps_d) > 1e-5:                       # away from the rounding edge
            assert info["dual"] == int(direct < eps_d), (t, direct)
        assert info["dual"] == int(info["delta_hat"] < eps_d), (t, info["delta_hat"])
        assert y_changed == bool(info["dual"])               # y-tilde moves only through the gate
        seen.add(info["dual"])
    assert seen == {0, 1}
    # a wrong power of eps_d or of K in the threshold would open the gate at another iteration
    first_open = next(t for t, info, _, _ in traj if info["dual"])
    assert first_open > 0 and traj[first_open - 1][2] >= eps_d > traj[first_open][2]


@pytest.mark.parametrize("T_min", [1, 10, 10 ** 6])
def test_stop_predicate_is_algorithm_1_break_line(T_min):
    """Algorithm 1's break: delta-hat < min(eps_d, eps_c), rho < eps_c and t + 1 >= T_min."""
    eps_d, eps_c = 0.05, 1e-4
    base = _trajectory_with_gate_crossing(eps_d, eps_c, T_min=1)
    t_ready = base[-1][0]                                     # first iteration whose tests all pass
    assert base[-1][1]["stop"] == 1 and t_ready + 1 > 1
    if T_min == 10 ** 6:
        T_min = t_ready + 3                                   # delays an otherwise-ready stop
    traj = _trajectory_with_gate_crossing(eps_d, eps_c, T_min, iters=t_ready + 10)
    for t, info, direct, _ in traj:
        want = info["delta_hat"] < min(eps_d, eps_c) and info["rho"] < eps_c and t + 1 >= T_min
        assert info["stop"] == int(want), (t, info)
    last_t = traj[-1][0]
    assert traj[-1][1]["stop"] == 1
    assert last_t + 1 >= T_min and last_t == max(t_ready, T_min - 1)


def test_descent_inequality_with_fixed_dual():
    """Corollary (descent): with y fixed and alpha < 1/L, each projected step lowers f-hat by at
    least (1 - alpha L) / (2 alpha) * ||U+ - U||_F^2."""
    _, Xhat, _, U, yt = _small_problem(n=120, d=5, r=3, seed=11)
    n, K, beta = U.shape[0], 3, 1.0
    y_norm = np.sqrt(n) * np.linalg.norm(yt.astype(np.float64))
    L = 2.0 + 2.0 * y_norm + beta * (6 * K + 2)
    alpha = 0.9 / L
    st = oracle.State(Xhat, U, yt)
    f_prev = oracle.objective(Xhat, st.U, yt, beta)
    for _ in range(60):
        Uprev = st.U.astype(np.float64).copy()
        info = st.step(K=K, alpha=alpha, beta=beta, eps_d=0.0, eps_c=0.0, T_min=1)
        assert info["dual"] == 0
        f_new = oracle.objective(Xhat, st.U, yt, beta)
        assert abs(info["fhat"] - f_prev) <= 1e-12 * max(1.0, abs(f_prev))
        move2 = np.sum((st.U.astype(np.float64) - Uprev) ** 2)
        assert f_new <= f_prev - (1 - alpha * L) / (2 * alpha) * move2 + 1e-7
        f_prev = f_new


def test_invariants_and_feasibility_progress():
    # random starts with r = K do not always reach the planted partition; this seed does
    spec = dataclasses.replace(synth.config(1).with_n(400), seed=1)
    X, lab, _ = synth.make_mixture(spec)
    hp = synth.default_hparams(spec.K)
    Xhat, _, _ = oracle.normalize(X)
    st = oracle.State(Xhat, synth.make_u0(spec.n, spec.K, spec.K, seed=1))
    rho0 = np.linalg.norm(st.q.astype(np.float64)) / np.sqrt(spec.n)
    rhos = []
    for _ in range(400):
        info = st.step(spec.K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], hp["T_min"])
        assert info["status"] == 0
        assert (st.U >= 0).all()
        assert abs(np.sum(st.U.astype(np.float64) ** 2) - spec.K) <= 1e-5
        if info["dual"]:
            rhos.append(info["rho"])
        if info["stop"]:
            break
    assert info["stop"] == 1
    assert rhos[-1] < 1e-4 < rho0 and rhos[-1] < 0.1 * rhos[0]
    # rows of a converged factor on well-separated data identify the planted groups
    pred = oracle.labels(st.U)
    best = max(np.mean(np.array(perm)[pred] == lab) for perm in itertools.permutations(range(spec.K)))
    assert best == 1.0


def test_planted_assignment_closed_forms():
    """H_ik = 1{i in G_k}/sqrt(|G_k|): ||H||_F^2 = K, g(H) = 0, ||H||_2 = 1, and
    J(G) = ||X||_F^2 - ||X^T H||_F^2 (Eq. "partition")."""
    spec = synth.config(1).with_n(300)
    X, lab, _ = synth.make_mixture(spec)
    n, K = spec.n, spec.K
    sizes = np.bincount(lab, minlength=K)
    H = np.zeros((n, K), np.float64)
    H[np.arange(n), lab] = 1.0 / np.sqrt(sizes[lab])
    H32 = H.astype(np.float32)
    p, q = oracle.residual(H32)
    np.testing.assert_allclose(p, np.sqrt(sizes), rtol=1e-6)
    assert np.abs(q).max() <= 5e-6
    assert abs(np.sum(H32.astype(np.float64) ** 2) - K) <= 1e-5
    assert abs(oracle.sym_eig_max(H.T @ H) - 1.0) <= 1e-12
    # cost identity, through the oracle's objective on the normalized data (y = 0, q = 0):
    Xhat, a, mean = oracle.normalize(X)
    f0 = oracle.objective(Xhat, H32, np.zeros(n, np.float32), beta=1.0)
    Xc = X.astype(np.float64) - mean
    J_identity = np.sum(Xc ** 2) + a * a * f0
    J_direct = oracle.kmeans_cost(X, lab, K)
    assert abs(J_identity - J_direct) <= 2e-5 * J_direct
    J_numpy = sum(np.sum((X[lab == k].astype(np.float64) - X[lab == k].astype(np.float64).mean(0)) ** 2)
                  for k in range(K))
    assert abs(J_direct - J_numpy) <= 1e-10 * J_numpy


def test_spectral_norm_against_library_and_closed_form():
    rng = np.random.default_rng(0)
    X = (rng.standard_normal((500, 9)) * rng.uniform(0.5, 4, size=9) + rng.uniform(-5, 5, size=9)).astype(np.float32)
    a, mean = oracle.spectral_norm(X, center=True)
    X64 = X.astype(np.float64)
    np.testing.assert_allclose(mean, X64.mean(0), rtol=1e-12, atol=1e-12)
    assert abs(a - np.linalg.norm(X64 - X64.mean(0), 2)) <= 1e-10 * a
    a0, mean0 = oracle.spectral_norm(X, center=False)
    assert (mean0 == 0).all() and abs(a0 - np.linalg.norm(X64, 2)) <= 1e-10 * a0
    # orthonormal columns scaled by (3, 2, 1): the spectral norm is 3
    Q, _ = np.linalg.qr(rng.standard_normal((64, 3)))
    Xo = (Q * np.array([3.0, 2.0, 1.0])).astype(np.float32)
    a1, _ = oracle.spectral_norm(Xo, center=False)
    assert abs(a1 - 3.0) <= 1e-6


def test_sym_eig_max_against_library():
    rng = np.random.default_rng(4)
    for d in (1, 2, 5, 17):
        B = rng.standard_normal((d, d))
        S = B + B.T - 3.0 * np.eye(d)
        assert abs(oracle.sym_eig_max(S) - np.linalg.eigvalsh(S)[-1]) <= 1e-10 * max(1.0, np.abs(S).max())
    assert oracle.sym_eig_max(np.diag([1.0, 7.0, -2.0])) == 7.0


def test_normalization_invariant_to_affine_rescaling():
    """X-hat does not change under X -> s X + 1 v^T (s > 0), so neither do the iterates."""
    rng = np.random.default_rng(8)
    X = rng.standard_normal((300, 6)).astype(np.float32)
    v = np.array([0.5, -1.0, 2.0, 0.25, -0.75, 4.0], np.float32)
    X2 = (4.0 * X + v).astype(np.float32)
    Xh1, a1, _ = oracle.normalize(X)
    Xh2, a2, _ = oracle.normalize(X2)
    assert abs(a2 - 4.0 * a1) <= 1e-5 * a2
    np.testing.assert_allclose(Xh1, Xh2, atol=2e-6 * np.abs(Xh1).max())
    assert abs(np.linalg.norm(Xh1.astype(np.float64), 2) - 1.0) <= 1e-6


def test_labels_tie_break_and_zero_rows():
    U = np.array([[0.0, 0.0, 0.0], [0.1, 0.3, 0.3], [0.5, 0.2, 0.5], [0.0, 0.0, 0.2]], np.float32)
    assert oracle.labels(U).tolist() == [0, 1, 0, 2]


def _brute_force_kmeans(X, K):
    """Exact K-means by enumerating every labelling of n <= 12 points."""
    X = X.astype(np.float64)
    n = X.shape[0]
    codes = np.arange(K ** n, dtype=np.int64)
    L = np.empty((codes.size, n), np.int8)
    for i in range(n):
        L[:, i] = codes % K
        codes //= K
    J = np.full(L.shape[0], np.sum(X ** 2))
    valid = np.ones(L.shape[0], bool)
    for k in range(K):
        M = (L == k)
        cnt = M.sum(1)
        valid &= cnt > 0
        S = M.astype(np.float64) @ X
        J -= np.sum(S ** 2, axis=1) / np.maximum(cnt, 1)
    J[~valid] = np.inf
    best = int(np.argmin(J))
    return L[best].astype(np.int32), float(J[best])


def _same_partition(a, b):
    pairs = set(zip(a.tolist(), b.tolist()))
    return len(pairs) == len(set(a.tolist())) == len(set(b.tolist()))


@pytest.mark.parametrize("K,seed", [(2, 0), (2, 1), (2, 2), (3, 0), (3, 1), (3, 2)])
def test_recovers_brute_force_optimum_on_tiny_mixtures(K, seed):
    X, planted = synth.separated_tiny_mixture(12, K, seed=seed)
    best, Jbest = _brute_force_kmeans(X, K)
    assert _same_partition(best, planted)           # the mixture is separated enough
    assert abs(oracle.kmeans_cost(X, best, K) - Jbest) <= 1e-9 * max(1.0, Jbest)
    Xhat, _, _ = oracle.normalize(X)
    U0 = synth.make_u0(12, K, K, seed=seed)
    U, _, info, iters, rc = oracle.run(Xhat, U0, K, alpha=0.1, beta=1.0, eps_d=0.05, eps_c=1e-4,
                                       T=5000, T_min=10)
    assert rc == 0 and info["stop"] == 1 and iters < 5000
    pred = oracle.labels(U)
    assert _same_partition(pred, best)
    assert abs(oracle.kmeans_cost(X, pred, K) - Jbest) <= 1e-9 * max(1.0, Jbest)


def test_breakdown_is_reported():
    """A step so large that every entry turns negative gives W = 0 and the breakdown status;
    U then holds the unscaled W (all zeros)."""
    X, _ = synth.separated_tiny_mixture(9, 3, seed=0)
    Xhat, _, _ = oracle.normalize(X)
    st = oracle.State(Xhat, synth.make_u0(9, 3, 3))
    info = st.step(K=3, alpha=50.0, beta=1.0, eps_d=0.05, eps_c=1e-4, T_min=10)
    assert info["status"] == -4 and info["a"] == 0.0
    assert (st.U == 0).all() and st.t == 0


def test_run_equals_repeated_steps():
    spec = synth.config(1).with_n(256)
    X, _, _ = synth.make_mixture(spec)
    hp = synth.default_hparams(spec.K)
    Xhat, _, _ = oracle.normalize(X)
    U0 = synth.make_u0(spec.n, spec.K, spec.K)
    U, yt, info, iters, rc = oracle.run(Xhat, U0, spec.K, hp["alpha"], hp["beta"], hp["eps_d"],
                                        hp["eps_c"], 25, hp["T_min"])
    st = oracle.State(Xhat, U0)
    for _ in range(25):
        last = st.step(spec.K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], hp["T_min"])
    assert iters == 25 and rc == 0
    assert np.array_equal(U, st.U) and np.array_equal(yt, st.ytilde)
    assert last["delta_hat"] == info["delta_hat"] and last["rho"] == info["rho"]


def test_numpy_iteration_matches_the_c_oracle():
    """The row-chunked numpy restatement used for the largest shape agrees with the C oracle entry by
    entry (two consecutive iterations, the second with a pending dual step)."""
    from oracle import np_iteration
    n, d, K = 3001, 24, 7
    spec = synth.MixtureSpec("t", n, d, K, "equal", 16.0, "unit", 10, 3)
    X, _, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    U0 = synth.make_u0(n, K, K, seed=3)
    hp = dict(synth.default_hparams(K), eps_d=10.0)           # gate always open: the dual step is exercised
    st = oracle.State(Xhat, U0)
    U, yt, dual = U0, np.zeros(n, np.float32), False
    for _ in range(2):
        ref = st.step(K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 100)
        U, yt, info = np_iteration.iteration(Xhat, U, yt, K, hp["alpha"], hp["beta"], hp["eps_d"], dual_pending=dual,
                                             rows=1000)
        dual = bool(info["dual"])
        assert np.abs(U.astype(np.float64) - st.U).max() <= 2e-7 * np.abs(st.U).max()
        for k in ("a", "b", "h", "fhat"):
            assert abs(info[k] - ref[k]) <= (1e-7 if k == "fhat" else 1e-9) * max(abs(ref[k]), 1e-3), (k, info[k], ref[k])
        assert abs(info["c"] - ref["c"]) <= 1e-7 * ref["c"] and abs(info["delta_hat"] - ref["delta_hat"]) <= 1e-9
        assert info["dual"] == ref["dual"] == 1


# ---- data-informed starting factor (appendix "Additional Computation Details", "Initialization") ----
def _init_problem(n=400, seed=1):
    spec = dataclasses.replace(synth.config(1).with_n(n), seed=seed)
    X, lab, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    Z = np.random.default_rng([seed, 77]).standard_normal((n, spec.K)).astype(np.float32)
    return spec, Xhat, Z, lab


def test_range_init_is_the_q_factor_of_the_sampled_range():
    from oracle import range_init
    spec, Xhat, Z, _ = _init_problem()
    U0, info = range_init.range_init(Xhat, Z, spec.K)
    Q = info["Q"]
    r = Z.shape[1]
    assert np.abs(Q.T @ Q - np.eye(r)).max() <= 1e-10          # orthonormal columns
    # the same basis as a Householder QR of the explicit n x n product, up to its sign convention
    X64 = Xhat.astype(np.float64)
    V = X64 @ (X64.T @ Z.astype(np.float64))
    Qh, Rh = np.linalg.qr(V)
    sign = np.sign(np.diag(Rh))
    assert np.abs(Q - Qh * sign).max() <= 1e-9
    assert np.abs(info["R"] - Rh * sign[:, None]).max() <= 1e-9 * np.abs(Rh).max()
    # projection onto {U >= 0, ||U||_F^2 = K}: the nonnegative part, rescaled (closest feasible point)
    W = np.maximum(Q, 0.0)
    ref = np.sqrt(spec.K) * W / np.linalg.norm(W)
    assert (U0 >= 0).all() and abs(np.sum(U0.astype(np.float64) ** 2) - spec.K) <= 1e-5
    np.testing.assert_allclose(U0, ref, atol=2e-7 * np.abs(ref).max())
    # among feasible points none is closer to Q than the projection (spot check against random feasible points)
    rng = np.random.default_rng(0)
    dist0 = np.linalg.norm(ref - Q)
    for _ in range(20):
        Y = np.abs(rng.standard_normal(Q.shape))
        Y *= np.sqrt(spec.K) / np.linalg.norm(Y)
        assert np.linalg.norm(Y - Q) >= dist0


def test_range_init_lowers_the_initial_objective():
    """The paper reports that the orthonormalized, data-informed start substantially lowers the initial
    augmented-Lagrangian value compared with a structure-free start."""
    from oracle import range_init
    better = 0
    for seed in (0, 1, 2, 3):
        spec, Xhat, Z, _ = _init_problem(seed=seed)
        U0, _ = range_init.range_init(Xhat, Z, spec.K)
        y0 = np.zeros(spec.n, np.float32)
        f_init = oracle.objective(Xhat, U0, y0, beta=1.0)
        f_unif = oracle.objective(Xhat, synth.make_u0(spec.n, spec.K, spec.K, seed=seed), y0, beta=1.0)
        better += f_init < f_unif
    assert better == 4


def test_range_init_needs_a_full_rank_sample():
    from oracle import range_init
    rng = np.random.default_rng(3)
    Xhat, _, _ = oracle.normalize(rng.standard_normal((200, 5)).astype(np.float32))
    Z = rng.standard_normal((200, 8)).astype(np.float32)          # r > d: V has rank <= d
    with pytest.raises(np.linalg.LinAlgError):
        range_init.range_init(Xhat, Z, 8)


# ---- label read-out for r > K (appendix "Additional Computation Details", "Recover cluster labels") ----
def _planted_factor_with_split_columns(n=600, K=4, per=3, seed=0, noise=0.0):
    """U >= 0 with r = per * K columns whose rows are constant within each planted cluster, every cluster's mass
    spread over its own `per` columns with different weights: U U^T is the planted block matrix."""
    rng = np.random.default_rng(seed)
    sizes = np.full(K, n // K)
    sizes[: n - sizes.sum()] += 1
    lab = np.repeat(np.arange(K), sizes)
    rng.shuffle(lab)
    r = per * K
    U = np.zeros((n, r))
    for k in range(K):
        w = rng.uniform(0.2, 1.0, size=per)
        w /= np.linalg.norm(w)
        U[np.ix_(lab == k, np.arange(per * k, per * (k + 1)))] = w / np.sqrt(sizes[k])
    if noise:
        U = np.abs(U + noise * rng.standard_normal(U.shape) / np.sqrt(n))
    return U.astype(np.float32), lab


def test_spectral_labels_recover_a_partition_that_row_argmax_splits():
    from oracle import spectral_labels as sl
    U, lab = _planted_factor_with_split_columns()
    labels, Y, passes = sl.spectral_labels(U, 4)
    assert _same_partition(labels, lab.astype(np.int32))
    # the row argmax is a valid column index but not a cluster index when r > K: the heaviest of a cluster's own
    # columns wins for all of its rows here, so the argmax only names K of the 12 columns
    assert set(oracle.labels(U).tolist()) <= set(range(12)) and len(set(oracle.labels(U).tolist())) == 4
    Un, _ = _planted_factor_with_split_columns(noise=0.3, seed=3)
    labels_n, _, _ = sl.spectral_labels(Un, 4)
    assert _same_partition(labels_n, _planted_factor_with_split_columns(seed=3)[1].astype(np.int32))


def test_spectral_embedding_distances_match_the_gram_route():
    """Leading left singular vectors from the r x r Gram matrix: P_K = U Q_K S_K^{-1} with U^T U = Q S^2 Q^T.
    Rows of the two embeddings have the same pairwise distances (signs and in-eigenspace rotations drop out)."""
    from oracle import spectral_labels as sl
    U, _ = _planted_factor_with_split_columns(noise=0.5, seed=1)
    K = 4
    Y = sl.embedding(U, K)
    U64 = U.astype(np.float64)
    lam, Q = np.linalg.eigh(U64.T @ U64)
    Yg = U64 @ (Q[:, ::-1][:, :K] / np.sqrt(lam[::-1][:K]))
    rng = np.random.default_rng(0)
    i, j = rng.integers(0, U.shape[0], 200), rng.integers(0, U.shape[0], 200)
    d_svd = np.linalg.norm(Y[i] - Y[j], axis=1)
    d_gram = np.linalg.norm(Yg[i] - Yg[j], axis=1)
    assert np.abs(d_svd - d_gram).max() <= 1e-9


def test_lloyd_ends_at_a_fixed_point_and_does_not_raise_the_cost():
    from oracle import spectral_labels as sl
    rng = np.random.default_rng(2)
    Y = np.concatenate([rng.standard_normal((80, 3)) + 4.0 * rng.standard_normal(3) for _ in range(5)])
    seeds = sl.farthest_point_seeds(Y, 5)
    assert len(set(seeds.tolist())) == 5 and seeds[0] == int(np.argmax((Y ** 2).sum(1)))
    # each seed is the farthest row from the seeds before it
    for m in range(1, 5):
        dmin = np.min(((Y[:, None, :] - Y[seeds[:m]][None]) ** 2).sum(2), axis=1)
        assert dmin[seeds[m]] == dmin.max()
    labels, centres, passes = sl.lloyd(Y, Y[seeds].copy(), max_iter=100)
    assert passes < 100
    d2 = ((Y[:, None, :] - centres[None]) ** 2).sum(2)
    assert np.array_equal(labels, np.argmin(d2, axis=1))
    for k in range(5):
        np.testing.assert_allclose(centres[k], Y[labels == k].mean(0), atol=1e-12)
    cost = lambda lab, C: float(((Y - C[lab]) ** 2).sum())
    lab0 = np.argmin(((Y[:, None, :] - Y[seeds][None]) ** 2).sum(2), axis=1)
    assert cost(labels, centres) <= cost(lab0, Y[seeds]) + 1e-12
