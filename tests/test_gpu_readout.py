"""GPU parity of the spectral label read-out for r >= K (gem_nlr_labels_spectral) against its oracle."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2609_36074_b200 as gem
from oracle import spectral_labels as sl
from gpu_helpers import make_solver

pytestmark = pytest.mark.gpu


def _planted(n, K, per, seed, noise):
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
    return U.astype(np.float32), lab.astype(np.int32)


def _same_partition(a, b):
    pairs = set(zip(a.tolist(), b.tolist()))
    return len(pairs) == len(set(a.tolist())) == len(set(b.tolist()))


def _solver_for(U, K, d=8):
    n = U.shape[0]
    X = np.random.default_rng(0).standard_normal((n, d)).astype(np.float32)
    Xhat, _, _ = oracle.normalize(X)
    return make_solver(Xhat, U, K, synth.default_hparams(K))


# (n, K, columns per cluster, noise): one and several tiles, odd r (bye round of the Jacobi pairing), larger K
@pytest.mark.parametrize("n,K,per,noise", [(600, 4, 3, 0.0), (5003, 4, 3, 0.3), (4100, 5, 1, 0.2), (20000, 20, 3, 0.3),
                                           (3001, 3, 7, 0.1), (70000, 8, 2, 0.3)])
def test_spectral_labels_match_oracle(n, K, per, noise):
    U, lab = _planted(n, K, per, seed=n % 7, noise=noise)
    s = _solver_for(U, K)
    rc, out, passes = s.labels_spectral(max_iter=50)
    assert rc == gem.OK, (rc, s.last_error())
    got = out.cpu().numpy()
    ref, Y, ref_passes = sl.spectral_labels(U, K, max_iter=50)
    assert got.min() >= 0 and got.max() < K
    assert _same_partition(got, lab) and _same_partition(ref, lab)
    assert _same_partition(got, ref)
    if noise:                                             # without noise all rows of a cluster coincide and the seeds tie
        assert np.array_equal(got, ref)                   # same seeds in the same order, same assignment
        assert passes == ref_passes
    # reproducible
    rc2, out2, _ = s.labels_spectral(max_iter=50)
    assert rc2 == gem.OK and torch.equal(out, out2)
    s.destroy()


def test_spectral_labels_after_a_run_with_three_columns_per_cluster():
    """The paper's setting r = 3 K: iterate from the data-informed start, then read the labels out both ways.  The
    two sides cluster the same factor (the GPU's); they may differ on rows that sit between two centres."""
    spec = synth.config(1)
    X, lab, _ = synth.make_mixture(spec)
    Xhat, _, _ = oracle.normalize(X)
    K, r = spec.K, 3 * spec.K
    Z = np.random.default_rng(5).standard_normal((spec.n, r)).astype(np.float32)
    hp = synth.default_hparams(K)
    s = make_solver(Xhat, Z, K, hp, T=300)
    assert s.init_range() == gem.OK
    rc, info, iters = s.run()
    assert rc >= 0
    Ug = s.U.cpu().numpy()
    rc, out, passes = s.labels_spectral()
    assert rc == gem.OK
    got = out.cpu().numpy()
    ref, _, _ = sl.spectral_labels(Ug, K)
    best = max(np.mean(np.array(perm)[got] == ref) for perm in itertools.permutations(range(K)))
    assert best >= 0.995, best
    s.destroy()


def test_spectral_labels_argument_errors_and_rank_deficiency():
    U, _ = _planted(3000, 4, 2, seed=1, noise=0.0)
    s = _solver_for(U, 4)
    out = torch.empty(3000, dtype=torch.int32, device="cuda")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    lib = gem.lib()
    assert lib.gem_nlr_labels_spectral(s._h, out.data_ptr(), small.data_ptr(), 1024, 10, None) == gem.E_WORKSPACE
    assert lib.gem_nlr_labels_spectral(s._h, out.data_ptr(), None, 0, 10, None) == gem.E_INVALID
    s.destroy()
    # a factor of rank 2 cannot give 4 singular vectors
    Ud = np.zeros((3000, 8), np.float32)
    Ud[:1500, 0] = 1.0
    Ud[1500:, 1] = 1.0
    s = _solver_for(Ud, 4)
    rc, _, _ = s.labels_spectral()
    assert rc == gem.E_BREAKDOWN
    s.destroy()
